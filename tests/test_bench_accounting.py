"""bench.py's work accounting against the oracle: the contexts and nodes that Algorithm 1's loop reaches,
computed from a call's outputs (accept length, accepted path), equal what the oracle actually tested."""
import numpy as np
import torch

import bench
import lantern_inputs as li
import oracle


def _check(inp, table, delta):
    res = oracle.verify_inputs(inp, table, delta)
    par = None if inp.tree_parents is None else torch.from_numpy(inp.tree_parents)
    ctx, nodes = bench.method_work(par, torch.from_numpy(res.accept_len), torch.from_numpy(res.accept_path), inp.N)
    assert nodes == int(res.tested.sum())
    # contexts = distinct parent contexts of the tested nodes
    want = 0
    for b in range(inp.B):
        parents = (np.arange(inp.N) - 1) if inp.tree_parents is None else inp.tree_parents[b]
        want += len({int(parents[i]) for i in range(inp.N) if res.tested[b, i]})
    assert ctx == want
    return ctx, nodes


def test_method_work_matches_the_oracle_on_chains_and_trees():
    V, k = 256, 12
    table = oracle.build_neighbors(li.codebook_gaussian(V, 4, seed=3), k)[0]
    chain = li.verify_inputs(40, 6, V, dtype=li.F32, has_uncond=False, cfg_scale=1.0, sigma_draft=0.8, seed=5)
    ctx, nodes = _check(chain, table, 0.2)
    assert ctx == nodes and 40 <= ctx <= 40 * 6
    tree = li.verify_inputs(30, 25, V, dtype=li.F32, has_uncond=False, cfg_scale=1.0, sigma_draft=1.0,
                            parents=li.tree_parents(30, 25, depth=4, seed=2), seed=6)
    ctx, nodes = _check(tree, table, 0.1)
    assert nodes >= ctx >= 30


def test_work_bytes():
    cfg = li.CONFIGS["batch_chain"]
    assert bench.context_bytes(cfg) == 3 * 16384 * 2 and bench.context_bytes(cfg, greedy=True) == 2 * 16384 * 2
    assert bench.work_bytes(cfg, 10, 12) == 10 * 98304 + 12 * 4000
