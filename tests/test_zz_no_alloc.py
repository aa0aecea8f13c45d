"""lantern_verify_static -- the entry point for callers that may not allocate device memory.

Some users of this library verify drafts at a point where a cudaMalloc is off the table: the
serving process gave all of its HBM to the KV cache and activation arenas at start-up, or the
step is latency-critical and cannot take the device-wide synchronisation an allocation brings.
For them the library keeps a fixed 6 MiB scratch array inside its own device image.  This test
calls that entry point through the C ABI and checks that it returns exactly what the ordinary
entry point (caller-supplied workspace) returns, on two calls in a row with different inputs --
the second call finds the first call's leftovers in the shared array and must not be disturbed
by them.  It also checks that a call too large for the fixed array is refused with a clear error,
that greedy decoding (T = 0) goes through the same entry point, and that a warmed-up call leaves the
device's free memory exactly where it was.

The file is named so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

import lantern_inputs as li
import oracle
import paper_2410_03355_b200 as lt
from parity import to_device

pytestmark = pytest.mark.gpu


def _outputs(B, N):
    i32 = dict(dtype=torch.int32, device="cuda")
    f32 = dict(dtype=torch.float32, device="cuda")
    return lt.VerifyOutputs(accept_len=torch.full((B,), -7, **i32), next_token=torch.full((B,), -7, **i32),
                            accept_path=torch.full((B, N), -7, **i32), status=torch.full((B,), -7, **i32),
                            node_qa=torch.zeros((B, N), **f32), node_px=torch.zeros((B, N), **f32),
                            node_m=torch.full((B, N), -7, **i32))


def _same(a: lt.VerifyOutputs, b: lt.VerifyOutputs):
    for f in ("accept_len", "next_token", "accept_path", "status"):
        assert torch.equal(getattr(a, f), getattr(b, f)), f
    # Per-node values: same kernels, same inputs, so a node evaluated in both calls carries bit-identical
    # values (NaN marks a node a call did not evaluate; which nodes off the accepted path get evaluated
    # ahead of time may differ from call to call).  Every node on the accepted path is evaluated in both.
    both = ~torch.isnan(a.node_qa) & ~torch.isnan(b.node_qa)
    for f in ("node_qa", "node_px", "node_m"):
        assert torch.equal(getattr(a, f)[both], getattr(b, f)[both]), f
    on_path = a.accept_path >= 0
    rows = torch.arange(a.accept_path.shape[0], device=a.accept_path.device)[:, None].expand_as(a.accept_path)
    assert bool(both[rows[on_path], a.accept_path[on_path].long()].all())


def test_static_workspace_matches_workspace_call_twice_in_a_row():
    V, k, delta = 2048, 100, 0.3
    table = torch.from_numpy(oracle.build_neighbors(li.codebook_gaussian(V, 8, seed=41), k)[0]).cuda()
    calls = [
        # a tree call first, then a larger chain call of a different shape that reuses the same scratch
        li.verify_inputs(16, 20, V, dtype=li.BF16, has_uncond=True, cfg_scale=3.0, rho=0.9, sigma_draft=1.0,
                         parents=li.tree_parents(16, 20, depth=4, seed=1), seed=51),
        li.verify_inputs(96, 5, V, dtype=li.BF16, has_uncond=True, cfg_scale=3.0, rho=0.9, sigma_draft=1.0,
                         peaked_frac=0.1, seed=52),
    ]
    for inp in calls:
        d = to_device(inp)
        want = lt.verify(d["target_logits"], d["draft_logits"], inp.cfg_scale, inp.T, d["draft_tokens"],
                         d["tree_parents"], table, delta, d["uniforms"], trace=True)
        torch.cuda.synchronize()
        got = lt.verify_static(d["target_logits"], d["draft_logits"], inp.cfg_scale, inp.T, d["draft_tokens"],
                               d["tree_parents"], table, delta, d["uniforms"], out=_outputs(inp.B, inp.N))
        torch.cuda.synchronize()
        _same(got, want)
        assert int(want.accept_len.sum()) > 0 and int((want.next_token >= 0).sum()) == inp.B
        # and both agree with the oracle on this input (decisions away from thresholds)
        ref = oracle.verify_inputs(inp, table.cpu().numpy(), delta)
        clear = (np.where(ref.tested.astype(bool), ref.margin, np.inf).min(axis=1) > 1e-6) & (ref.draw_margin > 1e-6)
        assert np.array_equal(got.accept_len.cpu().numpy()[clear], ref.accept_len[clear])
        assert np.array_equal(got.next_token.cpu().numpy()[clear], ref.next_token[clear])


def test_static_workspace_refuses_calls_beyond_its_size():
    V, k = 64, 4
    table = torch.from_numpy(oracle.build_neighbors(li.codebook_gaussian(V, 4, seed=42), k)[0]).cuda()
    B, N = 4096, 60                       # needs several times the fixed 6 MiB of scratch
    assert lt.verify_workspace_bytes(B, N, V, k) > lt.STATIC_WORKSPACE_BYTES
    tl = torch.zeros((1, B, N + 1, V), dtype=torch.bfloat16, device="cuda")
    dl = torch.zeros((B, N + 1, V), dtype=torch.bfloat16, device="cuda")
    tok = torch.zeros((B, N), dtype=torch.int32, device="cuda")
    un = torch.full((B, N + 1), 0.5, dtype=torch.float32, device="cuda")
    out = _outputs(B, N)
    with pytest.raises(lt.LanternError) as e:
        lt.verify_static(tl, dl, 1.0, 1.0, tok, None, table, 0.1, un, out=out)
    assert e.value.code == -4 and "workspace" in str(e.value)
    torch.cuda.synchronize()
    assert int(out.accept_len[0]) == -7   # nothing ran
    # the largest documented shapes do fit
    assert lt.verify_workspace_bytes(8192, 7) <= lt.STATIC_WORKSPACE_BYTES
    assert lt.verify_workspace_bytes(1024, 60) <= lt.STATIC_WORKSPACE_BYTES


def test_static_workspace_greedy_and_no_allocation():
    """T = 0 through the fixed array gives what the workspace call gives, and the call allocates nothing:
    the device's free memory is the same before and after a call that has run once before."""
    V, k, delta = 2048, 100, 0.3
    table = torch.from_numpy(oracle.build_neighbors(li.codebook_gaussian(V, 8, seed=41), k)[0]).cuda()
    inp = li.verify_inputs(40, 6, V, dtype=li.BF16, has_uncond=True, cfg_scale=3.0, rho=0.9, sigma_draft=0.5, seed=53)
    d = to_device(inp)
    want = lt.verify(d["target_logits"], None, inp.cfg_scale, 0.0, d["draft_tokens"], None, table, delta, None,
                     trace=True)
    out = _outputs(inp.B, inp.N)
    lt.verify_static(d["target_logits"], None, inp.cfg_scale, 0.0, d["draft_tokens"], None, table, delta, None,
                     out=out)
    torch.cuda.synchronize()
    _same(out, want)
    assert int(want.accept_len.sum()) > 0
    for T, dl, un in ((0.0, None, None), (1.0, d["draft_logits"], d["uniforms"])):
        lt.verify_static(d["target_logits"], dl, inp.cfg_scale, T, d["draft_tokens"], None, table, delta, un, out=out)
        torch.cuda.synchronize()
        free0 = torch.cuda.mem_get_info()[0]
        lt.verify_static(d["target_logits"], dl, inp.cfg_scale, T, d["draft_tokens"], None, table, delta, un, out=out)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free0
