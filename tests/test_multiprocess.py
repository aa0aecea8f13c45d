"""The multi-rank part of the benchmark, on CPU with the gloo backend (world size 2).

The verification path shards by sequence with no exchange step, so the only cross-rank logic
is: every rank draws its own batch (distinct seeds), times itself, and the job's figure uses
the maximum time over ranks.  This test runs that logic as two real processes.
"""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import lantern_inputs as li
    seed = bench.rank_seed(li.BASE_SEED, rank)
    inp = li.config_verify_inputs("tiny", B=2, V=64, seed=seed)
    # each rank "measures" a different time; the job must see the slower one on every rank
    times = bench.max_over_ranks([10.0 + rank, 3.0 - rank], dist, "cpu")
    dist.barrier()
    out[rank] = (seed, int(inp.draft_tokens.sum()), float(inp.target_logits.sum()), times,
                 bench.aggregate_rate(world, 4, 7, times[0]))
    dist.destroy_process_group()


def test_two_ranks_gloo():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    port = 29500 + (os.getpid() % 2000)
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    a, b = out[0], out[1]
    assert a[0] != b[0] and a[2] != b[2]              # different seeds, different batches
    assert a[3] == b[3] == [11.0, 3.0]                # max over ranks, identical on both
    assert a[4] == b[4] == pytest.approx(2 * 4 * 7 / 11.0e-3)


def test_single_rank_helpers_need_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert bench.rank_seed(100, 0) == 100 and bench.rank_seed(100, 3) != bench.rank_seed(100, 2)
