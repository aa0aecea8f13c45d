"""Seeded random sweep of the verification call against the oracle: shapes, storage types, guidance,
temperature, chain / tree, bound (TVD / JSD), top-k filter, greedy decoding and masked (-inf) tokens in
random combination.  Comparison rules are those of tests/parity.py and tests/test_gpu_greedy.py."""
import numpy as np
import pytest
import torch

import lantern_inputs as li
import oracle
from parity import assert_parity, compare, run_gpu
from test_gpu_greedy import check as greedy_check

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", [11, 12, 13, 14])
def test_random_combinations(seed):
    rng = np.random.default_rng(seed)
    for case in range(12):
        V = int(rng.choice([8, 64, 256, 520, 1000, 2048, 3000, 4096, 8192]))
        k = int(min(V, rng.choice([1, 2, 5, 16, 33, 100, 257, 600])))
        N, B = int(rng.integers(0, 13)), int(rng.integers(1, 20))
        dtype, unc = int(rng.choice([li.F32, li.BF16])), bool(rng.integers(2))
        T = float(rng.choice([1.0, 1.0, 0.7, 1.6]))
        delta = float(rng.choice([0.0, 0.02, 0.1, 0.3, 0.69, 1.5]))
        div = int(rng.choice([oracle.DIV_TVD, oracle.DIV_JSD]))
        top_k = int(rng.choice([0, 0, 1, 3, V // 3 + 1, V - 1, V, 1000]))
        tree = bool(rng.integers(2)) and N > 1
        greedy = bool(rng.integers(4) == 0)
        sd = float(rng.choice([0.3, 0.8, 1.5]))
        cfg = float(rng.choice([1.5, 3.0, 7.5])) if unc else 1.0
        gen = [li.codebook_gaussian, li.codebook_clustered, li.codebook_integer][int(rng.integers(3))]
        host = oracle.build_neighbors(gen(V, int(rng.choice([2, 8, 40])), seed=int(rng.integers(1000))), k)[0]
        dev = torch.from_numpy(host).cuda()
        par = li.tree_parents(B, N, depth=max(1, min(5, N)), seed=int(rng.integers(1000))) if tree else None
        inp = li.verify_inputs(B, N, V, dtype=dtype, has_uncond=unc, cfg_scale=cfg, T=T, sigma_target=1.0,
                               sigma_draft=sd, rho=float(rng.choice([0.0, 0.9])), parents=par,
                               seed=int(rng.integers(100000)))
        if rng.integers(3) == 0:      # masked tokens
            ninf = np.uint16(0xFF80) if dtype == li.BF16 else -np.inf
            m = rng.random(V) < 0.3
            inp.target_logits[..., m] = ninf
            if rng.integers(2):
                inp.draft_logits[..., m] = ninf
        what = dict(seed=seed, case=case, V=V, k=k, N=N, B=B, dtype=dtype, unc=unc, T=T, delta=delta, div=div,
                    top_k=top_k, tree=tree, greedy=greedy)
        try:
            if greedy:
                greedy_check(inp, host, dev, delta, divergence=div, top_k=top_k if top_k < V else 0)
            else:
                res = compare(inp, host, delta, run_gpu(inp, dev, delta, divergence=div, top_k=top_k),
                              divergence=div, top_k=top_k)
                assert_parity(res)
        except AssertionError as e:
            raise AssertionError(f"{what}: {e}") from e
