"""CUDA variants against the oracle: cosine neighbour metric (Section 5.3.1), JSD bound
(Section 5.3.2) and top-k logit filter (Appendix B.2) in sampling and in greedy decoding.  Comparison rules are those of
tests/parity.py and tests/test_gpu_greedy.py (the cut's window is in JSD units here)."""
import numpy as np
import pytest
import torch

import lantern_inputs as li
import oracle
import paper_2410_03355_b200 as lt
from parity import assert_parity, compare, run_gpu, tables
from test_gpu_greedy import check as greedy_check

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("V,D,k,kind", [(1024, 8, 16, "gaussian"), (777, 5, 100, "gaussian"), (2048, 8, 1000, "clustered"),
                                         (600, 256, 64, "clustered"), (512, 3, 512, "integer")])
def test_cosine_table(V, D, k, kind):
    gen = {"gaussian": li.codebook_gaussian, "clustered": li.codebook_clustered, "integer": li.codebook_integer}[kind]
    cb = gen(V, D, seed=13)
    rng = np.random.default_rng(1)
    cb = (cb * (2.0 ** rng.integers(-3, 4, size=(V, 1)))).astype(np.float32)    # lengths vary, directions do not
    if kind == "integer":
        cb[5] = 0.0                                                              # a zero code stays zero
    idx_o, dist_o = oracle.build_neighbors(cb, k, metric="cosine")
    idx_g, dist_g = lt.build_neighbors(torch.from_numpy(cb).cuda(), k, metric="cosine")
    torch.cuda.synchronize()
    assert np.array_equal(idx_g.cpu().numpy(), idx_o)
    assert np.array_equal(dist_g.cpu().numpy(), dist_o)
    # and the l2 entry point is untouched by the metric argument
    idx_l2 = lt.build_neighbors(torch.from_numpy(cb).cuda(), k, metric="l2")[0].cpu().numpy()
    assert np.array_equal(idx_l2, oracle.build_neighbors(cb, k)[0])
    assert not np.array_equal(idx_l2, idx_o)


@pytest.mark.parametrize("V,k,N,B,dtype,unc,delta", [
    (1024, 16, 4, 64, li.F32, False, 0.05),
    (1024, 16, 4, 64, li.BF16, True, 0.1),
    (1000, 300, 7, 40, li.BF16, True, 0.2),
    (8192, 1000, 5, 12, li.F32, True, 0.13),       # Table 3's matched JSD settings: 0.13 and 0.2
    (16384, 1000, 5, 24, li.BF16, True, 0.2),
    (2048, 2048, 2, 6, li.BF16, True, 0.7),        # above ln 2: the bound never binds
    (512, 32, 6, 50, li.BF16, True, 0.0),
])
def test_jsd_sampling_chains(V, k, N, B, dtype, unc, delta):
    cb = li.codebook_gaussian(V, 8, seed=31)
    inp = li.verify_inputs(B, N, V, dtype=dtype, has_uncond=unc, cfg_scale=3.0 if unc else 1.0, sigma_target=1.0,
                           sigma_draft=0.6, rho=0.9, seed=7 + V + k)
    host, dev = tables(cb, k, inp.draft_tokens)
    gpu = run_gpu(inp, dev, delta, divergence=oracle.DIV_JSD)
    res = compare(inp, host, delta, gpu, divergence=oracle.DIV_JSD)
    assert_parity(res)
    assert res["nodes_tested"] >= B
    if 0.0 < delta < 0.5:      # the JSD sets are strictly larger than the TVD sets at the same delta somewhere
        tv = run_gpu(inp, dev, delta)
        mj, mt = gpu.node_m.cpu().numpy()[:, 0], tv.node_m.cpu().numpy()[:, 0]
        assert (mj >= mt).all()
        if (mt < k - 1).sum() > 4:
            assert (mj > mt).any()


def test_jsd_sampling_trees():
    V, k = 2048, 64
    host = oracle.build_neighbors(li.codebook_clustered(V, 8, seed=5), k)[0]
    dev = torch.from_numpy(host).cuda()
    par = li.tree_parents(96, 30, depth=5, seed=3)
    inp = li.verify_inputs(96, 30, V, dtype=li.BF16, has_uncond=True, cfg_scale=3.0, sigma_target=1.0,
                           sigma_draft=1.0, rho=0.9, parents=par, seed=78)
    gpu = run_gpu(inp, dev, 0.1, divergence=oracle.DIV_JSD)
    res = compare(inp, host, 0.1, gpu, divergence=oracle.DIV_JSD)
    assert_parity(res)
    assert res["nodes_tested"] > 96 * 3      # sibling rounds (bounds on residual distributions) were exercised


@pytest.mark.parametrize("V,k,N,B,dtype,unc,delta", [
    (1024, 16, 4, 64, li.BF16, True, 0.1),
    (16384, 1000, 5, 24, li.BF16, True, 0.2),
    (8192, 1000, 5, 12, li.F32, True, 0.13),
])
def test_jsd_greedy(V, k, N, B, dtype, unc, delta):
    cb = li.codebook_gaussian(V, 8, seed=31)
    inp = li.verify_inputs(B, N, V, dtype=dtype, has_uncond=unc, cfg_scale=3.0, sigma_target=1.0,
                           sigma_draft=0.4, rho=0.9, seed=3 + V)
    host, dev = tables(cb, k, inp.draft_tokens)
    greedy_check(inp, host, dev, delta, divergence=oracle.DIV_JSD)


def test_bad_variant_arguments():
    V, k = 512, 8
    dev = torch.zeros((V, k), dtype=torch.int32, device="cuda")
    inp = li.verify_inputs(2, 2, V, seed=1)
    with pytest.raises(ValueError):
        run_gpu(inp, dev, 0.1, divergence=7) if False else lt.verify(None, None, 1.0, 1.0, None, None, dev, 0.1, None,
                                                                      divergence="kl")
    lib = lt.load_library()
    assert lib.lantern_build_workspace_bytes_metric(V, 8, k, 5) == 0
    assert lib.lantern_verify_workspace_bytes_ex(4, 4, V, k, 0, -1) == 0


# ------------------------------------------------------------------------------------ top-k filter
def _table(V, k, tokens):
    return tables(li.codebook_gaussian(V, 8, seed=31), k, tokens)


@pytest.mark.parametrize("V,k,N,B,dtype,unc,T,K,div", [
    (1024, 16, 4, 64, li.F32, False, 1.0, 100, oracle.DIV_TVD),
    (1024, 16, 4, 64, li.BF16, True, 1.0, 100, oracle.DIV_TVD),      # bf16: ties at the threshold are kept
    (1000, 300, 7, 40, li.BF16, True, 0.7, 37, oracle.DIV_TVD),      # temperature: thresholds on l / T
    (8192, 1000, 5, 12, li.F32, True, 1.0, 1000, oracle.DIV_JSD),
    (16384, 1000, 5, 24, li.BF16, True, 1.0, 1000, oracle.DIV_TVD),  # the text-conditional setting of Appendix B.2
    (16384, 1000, 5, 24, li.BF16, True, 1.0, 2000, oracle.DIV_JSD),
    (512, 32, 6, 50, li.BF16, True, 1.0, 1, oracle.DIV_TVD),         # K = 1: both distributions are point masses
    (512, 32, 6, 50, li.BF16, False, 1.0, 511, oracle.DIV_TVD),      # one token cut
    (512, 32, 6, 50, li.F32, False, 1.0, 512, oracle.DIV_TVD),       # K = V: filter off
    (8, 8, 3, 17, li.BF16, False, 1.0, 3, oracle.DIV_TVD),
])
def test_top_k_sampling(V, k, N, B, dtype, unc, T, K, div):
    inp = li.verify_inputs(B, N, V, dtype=dtype, has_uncond=unc, cfg_scale=3.0 if unc else 1.0, T=T, sigma_target=1.0,
                           sigma_draft=0.6, rho=0.9, seed=11 + V + K)
    host, dev = _table(V, k, inp.draft_tokens)
    gpu = run_gpu(inp, dev, 0.2, divergence=div, top_k=K)
    res = compare(inp, host, 0.2, gpu, divergence=div, top_k=K)
    assert_parity(res)
    assert res["nodes_tested"] >= (B if K > 1 else B // 4)     # (nodes of sequences without a status bit)
    # K = 1 makes target and drafter point masses: a drafted token outside their support leaves a residual
    # without weight, and the next token then comes from the context's own target (reported, and identical
    # on both sides)
    assert (res["degenerate"] > 0) == (K == 1)
    if K < V // 2:     # the filter matters: without it the decisions differ somewhere
        plain = oracle.verify_inputs(inp, host, 0.2, div)
        filt = oracle.verify_inputs(inp, host, 0.2, div, K)
        assert not (np.array_equal(plain.next_token, filt.next_token) and np.array_equal(plain.qa, filt.qa))


def test_top_k_trees_and_masked_logits():
    V, k, K = 2048, 64, 200
    host = oracle.build_neighbors(li.codebook_clustered(V, 8, seed=5), k)[0]
    dev = torch.from_numpy(host).cuda()
    par = li.tree_parents(96, 30, depth=5, seed=3)
    inp = li.verify_inputs(96, 30, V, dtype=li.BF16, has_uncond=True, cfg_scale=3.0, sigma_target=1.0,
                           sigma_draft=1.0, rho=0.9, parents=par, seed=79)
    neg_inf = np.uint16(0xFF80)
    inp.target_logits[:, 3, :, 100:1990] = neg_inf      # fewer than K tokens above -inf: nothing to cut
    inp.draft_logits[3, :, 100:1990] = neg_inf
    inp.target_logits[:, 4, :, ::3] = neg_inf           # masked tokens elsewhere
    gpu = run_gpu(inp, dev, 0.15, top_k=K)
    res = compare(inp, host, 0.15, gpu, top_k=K)
    assert_parity(res)
    assert res["nodes_tested"] > 96 * 3


@pytest.mark.parametrize("V,k,N,B,dtype,unc,K,div", [
    (1024, 16, 4, 64, li.BF16, True, 50, oracle.DIV_TVD),
    (16384, 1000, 5, 24, li.BF16, True, 1000, oracle.DIV_TVD),
    (8192, 1000, 5, 12, li.F32, True, 2000, oracle.DIV_JSD),
])
def test_top_k_greedy(V, k, N, B, dtype, unc, K, div):
    inp = li.verify_inputs(B, N, V, dtype=dtype, has_uncond=unc, cfg_scale=3.0, sigma_target=1.0,
                           sigma_draft=0.4, rho=0.9, seed=5 + V)
    host, dev = _table(V, k, inp.draft_tokens)
    greedy_check(inp, host, dev, 0.2, divergence=div, top_k=K)


def test_top_k_nan_rows_are_still_reported():
    V, k = 1024, 16
    inp = li.verify_inputs(12, 4, V, dtype=li.F32, has_uncond=False, cfg_scale=1.0, sigma_target=1.0,
                           sigma_draft=0.4, rho=0.9, seed=8)
    host, dev = _table(V, k, inp.draft_tokens)
    inp.target_logits[0, 3, 0, 17] = np.nan
    inp.draft_logits[6, 0, 5] = np.nan
    ora = oracle.verify_inputs(inp, host, 0.3, top_k=64)
    g = run_gpu(inp, dev, 0.3, top_k=64)
    assert np.array_equal(g.status.cpu().numpy(), ora.status) and ora.status[3] and ora.status[6]
    ok = ora.status == 0
    assert np.array_equal(g.accept_len.cpu().numpy()[ok], ora.accept_len[ok])
