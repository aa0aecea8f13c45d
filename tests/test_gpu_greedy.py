"""CUDA greedy-decoding verification (T = 0; Section 4.3, last sentence) against the oracle.

Rule: accept lengths, next tokens and accepted paths are identical to the oracle's, except where
a decision of the walk lies within WINDOW of flipping (|sum_A q - max_{x not in A} q| or the prefix
cut's distance to delta, both in probability units).  A sequence that differs is replayed node by
node with the oracle's per-row routines along the path the library took: every decision away from
the window must be the oracle's, a decision inside it may go either way, and the emitted token
must be the arg max of the context where that path ends.  sum_A q agrees to REL wherever the cut
agrees.
"""
import numpy as np
import pytest
import torch

import lantern_inputs as li
import oracle
import paper_2410_03355_b200 as lt
from parity import DIV_NAME, REL, WINDOW, tables, to_device

pytestmark = pytest.mark.gpu


def run_gpu(inp, table_dev, delta, trace=True, with_unused=False, divergence=oracle.DIV_TVD, top_k=0):
    d = to_device(inp)
    out = lt.verify(d["target_logits"], d["draft_logits"] if with_unused else None, inp.cfg_scale, 0.0,
                    d["draft_tokens"], d["tree_parents"], table_dev, delta,
                    d["uniforms"] if with_unused else None, trace=trace, divergence=DIV_NAME[divergence], top_k=top_k)
    torch.cuda.synchronize()
    return out


def replay(inp, table, delta, b, g_len, g_tok, g_path, divergence=oracle.DIV_TVD, top_k=0):
    """Is the library's (len, token, path) of sequence b a valid greedy walk up to WINDOW?"""
    N = inp.N
    par = inp.tree_parents[b] if inp.tree_parents is not None else np.arange(N) - 1
    cur, depth = 0, 0
    while True:
        ru = inp.target_logits[1, b, cur] if inp.has_uncond else None
        q = oracle.row_distribution(inp.target_logits[0, b, cur], ru, inp.dtype, inp.cfg_scale, 1.0, top_k)
        accepted = -1
        for c in [i for i in range(N) if par[i] == cur - 1]:
            x = inp.draft_tokens[b, c]
            m, moved, cut_margin = oracle.a_set(q, table[x], delta, divergence)
            qa = q[x] + moved
            mask = np.ones(inp.V, bool)
            mask[table[x, : m + 1]] = False
            outside = q[mask].max() if mask.any() else -1.0
            margin = min(abs(qa - outside), cut_margin if table.shape[1] > 1 else np.inf)
            took = depth < g_len and g_path[depth] == c
            if margin >= WINDOW and took != bool(qa >= outside):
                return False
            if took:
                accepted = c
                break
        if accepted < 0:
            return depth == g_len and g_tok == int(np.argmax(q))
        cur, depth = accepted + 1, depth + 1


def check(inp, host, dev, delta, divergence=oracle.DIV_TVD, top_k=0, **kw):
    gpu = run_gpu(inp, dev, delta, divergence=divergence, top_k=top_k, **kw)
    return check_outputs(inp, host, delta, gpu, divergence, top_k)


def check_outputs(inp, host, delta, gpu, divergence=oracle.DIV_TVD, top_k=0):
    ora = oracle.verify_greedy(inp.target_logits, inp.dtype, inp.cfg_scale, inp.has_uncond, inp.draft_tokens,
                               inp.tree_parents, host, delta, divergence, top_k)
    g_len, g_tok = gpu.accept_len.cpu().numpy(), gpu.next_token.cpu().numpy()
    g_path, g_st = gpu.accept_path.cpu().numpy(), gpu.status.cpu().numpy()
    assert np.array_equal(g_st, ora.status)
    near = 0
    for b in range(inp.B):
        if (g_len[b] == ora.accept_len[b] and g_tok[b] == ora.next_token[b]
                and np.array_equal(g_path[b], ora.accept_path[b])):
            continue
        assert replay(inp, host, delta, b, g_len[b], g_tok[b], g_path[b], divergence, top_k), \
            (b, g_len[b], ora.accept_len[b])
        near += 1
    assert near <= max(2, inp.B // 50), near
    qa, m = gpu.node_qa.cpu().numpy(), gpu.node_m.cpu().numpy()
    t = ora.tested.astype(bool) & (ora.status[:, None] == 0)
    far = t & (ora.margin >= WINDOW)
    assert np.array_equal(m[far], ora.m[far])
    agree = t & (m == ora.m)
    assert agree.sum() > 0 or not t.any()         # (no node tested at all: N = 0, or every sequence flagged)
    assert (np.abs(qa[agree] - ora.qa[agree]) <= REL * ora.qa[agree]).all()
    assert not gpu.node_px.cpu().numpy()[t].any()       # trace entries of untested nodes are not written
    return ora, near


@pytest.mark.parametrize("V,k,N,B,dtype,unc,delta", [
    (1024, 16, 4, 64, li.F32, False, 0.1),
    (1024, 16, 4, 64, li.BF16, True, 0.1),
    (8, 1, 1, 33, li.F32, False, 0.3),            # k = 1: plain greedy speculative decoding
    (8, 8, 3, 17, li.BF16, False, 0.5),
    (1000, 300, 7, 40, li.BF16, True, 0.2),       # V not a power of two
    (8192, 1000, 5, 12, li.F32, True, 0.1),
    (16384, 1000, 5, 12, li.F32, True, 0.1),      # greedy has no fp32 size limit below 16384
    (8200, 64, 3, 9, li.BF16, True, 0.05),
    (2048, 2048, 2, 6, li.BF16, True, 2.0),       # k = V, bound never reached: two scan rounds, A = everything
    (512, 32, 6, 50, li.BF16, True, 0.0),         # delta = 0: plain greedy
])
def test_chain_shapes(V, k, N, B, dtype, unc, delta):
    cb = li.codebook_gaussian(V, 8, seed=31)
    inp = li.verify_inputs(B, N, V, dtype=dtype, has_uncond=unc, cfg_scale=3.0 if unc else 1.0, sigma_target=1.0,
                           sigma_draft=0.4, rho=0.9, seed=101 + V + k)
    host, dev = tables(cb, k, inp.draft_tokens)
    ora, _ = check(inp, host, dev, delta)
    if delta >= 2.0:
        assert (ora.accept_len == N).all()        # sum over everything = 1 >= any q


def test_trees_and_sibling_order():
    V, k = 2048, 64
    host = oracle.build_neighbors(li.codebook_clustered(V, 8, seed=5), k)[0]
    dev = torch.from_numpy(host).cuda()
    par = li.tree_parents(96, 30, depth=5, seed=3)
    inp = li.verify_inputs(96, 30, V, dtype=li.BF16, has_uncond=True, cfg_scale=3.0, sigma_target=1.0,
                           sigma_draft=0.5, rho=0.9, parents=par, seed=77)
    ora, _ = check(inp, host, dev, 0.3)
    assert ora.accept_len.max() >= 2 and ora.tested.sum() > 96 * 2


def test_unused_inputs_are_ignored_and_no_nodes():
    V, k = 1024, 16
    host = oracle.build_neighbors(li.codebook_gaussian(V, 8, seed=31), k)[0]
    dev = torch.from_numpy(host).cuda()
    inp = li.verify_inputs(40, 5, V, dtype=li.BF16, has_uncond=True, cfg_scale=3.0, sigma_target=1.0,
                           sigma_draft=0.4, rho=0.9, seed=5)
    a = run_gpu(inp, dev, 0.2)
    b = run_gpu(inp, dev, 0.2, with_unused=True)
    for f in ("accept_len", "next_token", "accept_path", "status", "node_qa", "node_m"):
        assert torch.equal(getattr(a, f), getattr(b, f)), f
    # N = 0: the next token is the arg max of the only context
    inp0 = li.verify_inputs(25, 0, V, dtype=li.F32, has_uncond=False, cfg_scale=1.0, sigma_target=1.0,
                            sigma_draft=0.4, rho=0.9, seed=6)
    ora = oracle.verify_greedy(inp0.target_logits, inp0.dtype, 1.0, 0, inp0.draft_tokens, None, host, 0.2)
    g = run_gpu(inp0, dev, 0.2, trace=False)
    assert np.array_equal(g.next_token.cpu().numpy(), ora.next_token) and not g.accept_len.any()


def test_status_bits():
    V, k = 1024, 16
    host = oracle.build_neighbors(li.codebook_gaussian(V, 8, seed=31), k)[0]
    inp = li.verify_inputs(12, 4, V, dtype=li.F32, has_uncond=False, cfg_scale=1.0, sigma_target=1.0,
                           sigma_draft=0.4, rho=0.9, seed=8)
    inp.draft_tokens[1, 2] = V                      # bad token
    inp.target_logits[0, 3, 0, 17] = np.nan         # non-finite root context
    inp.target_logits[0, 5, 4, :] = -np.inf         # no finite logit at the leaf
    bad_table = host.copy()
    bad_table[inp.draft_tokens[7, 0], 1] = -5       # table entry out of range
    dev = torch.from_numpy(bad_table).cuda()
    ora = oracle.verify_greedy(inp.target_logits, inp.dtype, 1.0, 0, inp.draft_tokens, None, bad_table, 0.3)
    g = run_gpu(inp, dev, 0.3)
    assert np.array_equal(g.status.cpu().numpy(), ora.status)
    assert ora.status[1] and ora.status[3] and ora.status[7]
    bad = ora.status != 0
    assert np.array_equal(g.next_token.cpu().numpy()[bad & (ora.next_token < 0)], ora.next_token[bad & (ora.next_token < 0)])
    ok = ~bad
    assert np.array_equal(g.accept_len.cpu().numpy()[ok], ora.accept_len[ok])
    assert np.array_equal(g.next_token.cpu().numpy()[ok], ora.next_token[ok])


def test_bench_shape_sample():
    """The batch_chain shape (V = 16384, k = 1000, bf16 + guidance) at a batch the oracle finishes in seconds."""
    c = li.CONFIGS["batch_chain"]
    cb = li.config_codebook("batch_chain")
    inp = li.config_verify_inputs("batch_chain", step=0, B=48)
    host, dev = tables(cb, c["k"], inp.draft_tokens)
    check(inp, host, dev, c["delta"])


@pytest.mark.parametrize("workload,sample", [("batch_chain", 96), ("stress", 64)])
def test_bench_sized_call_against_sampled_oracle(workload, sample):
    """The call `bench.py --greedy` times, checked on a seeded sample of its sequences."""
    import bench
    import lantern_inputs.device as lid
    from test_gpu_fullsize import _oracle_rows, _properties, _table, _take
    w = bench.WORKLOADS[workload]
    cfg = li.CONFIGS[w["config"]]
    B, N, V, delta = w["B"], cfg["N"], cfg["V"], cfg["delta"]
    table = _table(w["config"])
    d = lid.config_verify_inputs_device(w["config"], B=B, seed=bench.rank_seed(li.BASE_SEED, 0))
    out = lt.verify(d["target_logits"], None, d["cfg_scale"], 0.0, d["draft_tokens"], d["tree_parents"], table,
                    delta, None, trace=True)
    torch.cuda.synchronize()
    _properties(d, out, N, V)
    rows = np.sort(np.random.default_rng(12).choice(B, size=min(sample, B), replace=False))
    host = lid.to_host(d, rows=rows)
    check_outputs(host, _oracle_rows(w["config"], host, table), delta, _take(out, rows))
    out2 = lt.verify(d["target_logits"], None, d["cfg_scale"], 0.0, d["draft_tokens"], d["tree_parents"], table,
                     delta, None)
    torch.cuda.synchronize()
    assert torch.equal(out.accept_len, out2.accept_len) and torch.equal(out.next_token, out2.next_token)
    assert torch.equal(out.accept_path, out2.accept_path)
