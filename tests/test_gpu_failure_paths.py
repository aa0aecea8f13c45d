"""Failure paths of the verification call on the GPU, made without any fault: a bounded wait that runs
out (the copy is withheld on purpose, nothing is in flight), a corrupt neighbour entry ahead of and
behind the slot that ends a set, a residual without weight, and the call-level summaries."""
import dataclasses

import numpy as np
import pytest
import torch

import lantern_inputs as li
import oracle
import paper_2410_03355_b200 as lt
from parity import assert_parity, compare, run_gpu, to_device

pytestmark = pytest.mark.gpu


def _call(d, inp, table, delta, ws=None):
    out = lt.verify(d["target_logits"], d["draft_logits"], inp.cfg_scale, inp.T, d["draft_tokens"],
                    d["tree_parents"], table, delta, d["uniforms"], workspace=ws)
    torch.cuda.synchronize()
    return out


def _setup(B, N, V=512, k=8, seed=3):
    host = oracle.build_neighbors(li.codebook_gaussian(V, 8, seed=36), k)[0]
    inp = li.verify_inputs(B, N, V, dtype=li.BF16, has_uncond=True, cfg_scale=2.0, rho=0.9, sigma_draft=0.6, seed=seed)
    return inp, to_device(inp), torch.from_numpy(host).cuda()


def _poisoned_workspace(B, N, V, k):
    ws = torch.empty(lt.verify_workspace_bytes(B, N, V, k), dtype=torch.uint8, device="cuda")
    ws.fill_(0x5a)           # whatever an earlier call may have left there must not leak into this one
    return ws


def test_a_wait_that_runs_out_flags_exactly_that_sequence():
    """Few contexts, one per consumer group: the copy of one root context is never started, its group's
    bounded wait runs out, the kernel returns, and INTERNAL is reported for that sequence alone."""
    B, N, bad = 16, 1, 5
    inp, d, table = _setup(B, N)
    want = _call(d, inp, table, 0.2)
    try:
        lt.debug_wait_test(max_tries=300, withhold_context=bad * (N + 1))
        ws = _poisoned_workspace(B, N, inp.V, table.shape[1])
        got = _call(d, inp, table, 0.2, ws)
        bits = lt.last_status(ws)
    finally:
        lt.debug_wait_test(0, -1)
    st = got.status.cpu().numpy()
    assert st[bad] == lt.ST_INTERNAL and int(got.next_token[bad]) == -1 and int(got.accept_len[bad]) == 0
    others = np.arange(B) != bad
    assert not st[others].any()
    for f in ("accept_len", "next_token", "accept_path"):
        assert torch.equal(getattr(got, f)[others], getattr(want, f)[others]), f
    assert bits == lt.ST_INTERNAL
    # the device is as usable as before
    again = _call(d, inp, table, 0.2)
    assert torch.equal(again.next_token, want.next_token) and not again.status.any()


def test_a_wait_that_runs_out_in_a_large_call():
    """Many contexts per group: the group that gives up takes the few contexts it had already drawn from
    the queue with it.  Every sequence is either reported (INTERNAL, no token, a valid accepted prefix) or
    carries exactly the result of the undisturbed call; nothing indexes out of range."""
    B, N, bad = 2048, 3, 777
    inp, d, table = _setup(B, N, seed=4)
    want = _call(d, inp, table, 0.2)
    try:
        lt.debug_wait_test(max_tries=3000, withhold_context=bad * (N + 1))
        got = _call(d, inp, table, 0.2, _poisoned_workspace(B, N, inp.V, table.shape[1]))
    finally:
        lt.debug_wait_test(0, -1)
    st = got.status.cpu().numpy()
    flagged = (st & lt.ST_INTERNAL) != 0
    assert flagged[bad] and 1 <= flagged.sum() <= 64, flagged.sum()
    assert not (st & ~lt.ST_INTERNAL).any()
    ok = ~flagged
    for f in ("accept_len", "next_token", "accept_path"):
        g, w = getattr(got, f).cpu().numpy(), getattr(want, f).cpu().numpy()
        assert np.array_equal(g[ok], w[ok]), f
    g_len, g_tok, g_path = (getattr(got, f).cpu().numpy() for f in ("accept_len", "next_token", "accept_path"))
    w_path = want.accept_path.cpu().numpy()
    for b in np.flatnonzero(flagged):
        assert g_tok[b] == -1 and 0 <= g_len[b] <= N
        assert np.array_equal(g_path[b, :g_len[b]], w_path[b, :g_len[b]]) and (g_path[b, g_len[b]:] == -1).all()


def test_corrupt_table_entry_before_and_after_the_cut():
    """A neighbour entry outside [0, V) is reported where Algorithm 2's loop meets it: ahead of the slot that
    ends the set, never behind it."""
    V, k, B, N, delta = 512, 64, 24, 2, 0.05
    cb = li.codebook_gaussian(V, 8, seed=37)
    host = oracle.build_neighbors(cb, k)[0]
    inp = li.verify_inputs(B, N, V, dtype=li.BF16, has_uncond=True, cfg_scale=2.0, rho=0.9, sigma_draft=0.6, seed=6)
    ora = oracle.verify_inputs(inp, host, delta)
    m0 = int(ora.m[0, 0])
    assert 2 <= m0 < k - 3, m0           # the first node's set ends inside the row
    x0 = int(inp.draft_tokens[0, 0])
    seen = set()
    for slot in (1, m0, m0 + 1, m0 + 2, k - 1):
        bad = host.copy()
        bad[x0, slot] = V + 7
        ref = oracle.verify_inputs(inp, bad, delta)
        gpu = run_gpu(inp, torch.from_numpy(bad).cuda(), delta)
        res = compare(inp, bad, delta, gpu, ora=ref)
        assert_parity(res)
        assert np.array_equal(gpu.status.cpu().numpy(), ref.status)
        seen.add((slot <= m0, bool(ref.status[0] & oracle.ST_BAD_TABLE)))
    assert (True, True) in seen and (False, False) in seen and (True, False) not in seen


def test_residual_without_weight_draws_from_the_target():
    """Target and drafter equal, the drafted token outside their support: the rejection leaves a residual of
    zero weight, which both sides report, and the next token comes from the context's own target."""
    V, k, B, N = 64, 4, 12, 2
    host = oracle.build_neighbors(li.codebook_gaussian(V, 4, seed=38), k)[0]
    inp = li.verify_inputs(B, N, V, dtype=li.F32, has_uncond=False, cfg_scale=1.0, sigma_draft=0.5, seed=8)
    inp.draft_logits[:] = inp.target_logits[0]
    for b in range(0, B, 2):
        x = int(inp.draft_tokens[b, 0])
        nb = host[x]
        inp.target_logits[0, b, 0, nb] = -np.inf           # neither the token nor its neighbours carry mass
        inp.draft_logits[b, 0, nb] = -np.inf
    ref = oracle.verify_inputs(inp, host, 0.3)
    assert (ref.status[0::2] == oracle.ST_DEGENERATE).all() and (ref.next_token[0::2] >= 0).all()
    assert (ref.accept_len[0::2] == 0).all()
    gpu = run_gpu(inp, torch.from_numpy(host).cuda(), 0.3)
    res = compare(inp, host, 0.3, gpu, ora=ref)
    assert_parity(res)
    assert res["near"] == 0
    assert np.array_equal(gpu.next_token.cpu().numpy(), ref.next_token)


def test_call_summaries():
    B, N = 300, 5
    inp, d, table = _setup(B, N, seed=9)
    ws = torch.empty(lt.verify_workspace_bytes(B, N, inp.V, table.shape[1]), dtype=torch.uint8, device="cuda")
    out = _call(d, inp, table, 0.2, ws)
    assert lt.last_status(ws) == 0
    c = lt.verify_counts(ws)
    assert c["contexts"] == B * N and c["evaluated"] + c["skipped"] == B * N
    # every context on an accepted path was evaluated: one per accepted node's parent, plus the one that stopped the walk
    al = out.accept_len.cpu().numpy()
    assert c["evaluated"] >= int(np.minimum(al + 1, N).sum())
    assert c["from_q"] == int((al == N).sum())
    bad = dataclasses.replace(inp, draft_tokens=inp.draft_tokens.copy())
    bad.draft_tokens[3, 1] = inp.V
    db = to_device(bad)
    _call(db, bad, table, 0.2, ws)
    assert lt.last_status(ws) == lt.ST_BAD_TOKEN
