"""CUDA neighbour-table builder against the oracle: indices and distances bit-exact."""
import numpy as np
import pytest
import torch

import lantern_inputs as li
import oracle
import paper_2410_03355_b200 as lt

pytestmark = pytest.mark.gpu


def _gpu(cb, k):
    idx, dist = lt.build_neighbors(torch.from_numpy(cb).cuda(), k)
    torch.cuda.synchronize()
    return idx.cpu().numpy(), dist.cpu().numpy()


@pytest.mark.parametrize("V,D,k", [(1024, 8, 16), (1000, 8, 1), (520, 3, 520), (64, 1, 7), (2048, 8, 300),
                                   (777, 5, 100), (300, 32, 33)])
def test_small_d_exact(V, D, k):
    cb = li.codebook_gaussian(V, D, seed=21, normalise=(D > 1))
    gi, gd = _gpu(cb, k)
    oi, od = oracle.build_neighbors(cb, k)
    assert np.array_equal(gi, oi)
    assert np.array_equal(gd.view(np.uint32), od.view(np.uint32))


def test_ties_and_duplicates_exact():
    # integer codebook: massive exact ties, broken by index; duplicates of a code keep self first
    cb = li.codebook_integer(1500, 4, lo=-2, hi=3, seed=5)
    cb[700] = cb[3]
    for k in (2, 64, 999):
        gi, gd = _gpu(cb, k)
        oi, od = oracle.build_neighbors(cb, k)
        assert np.array_equal(gi, oi), k
        assert np.array_equal(gd, od), k
    const = np.ones((600, 8), np.float32)          # every distance is 0: order is pure index order
    gi, _ = _gpu(const, 50)
    oi, _ = oracle.build_neighbors(const, 50)
    assert np.array_equal(gi, oi)


def test_outliers_and_overflowing_distances_exact():
    # One code far away stretches the key range so that every other key falls into the select's first bin
    # (the crowded-bin path with all of its passes); codes of magnitude 1e30 make distances overflow to inf
    # (equal keys, ordered by index).
    cb = li.codebook_gaussian(3000, 8, seed=77)
    cb[1234] *= 1e15
    for k in (5, 300, 3000):
        gi, gd = _gpu(cb, k)
        oi, od = oracle.build_neighbors(cb, k)
        assert np.array_equal(gi, oi), k
        assert np.array_equal(gd.view(np.uint32), od.view(np.uint32)), k
    cb = li.codebook_gaussian(900, 4, seed=78)
    cb[::7] *= 1e30
    with np.errstate(over="ignore"):
        gi, gd = _gpu(cb, 200)
        oi, od = oracle.build_neighbors(cb, 200)
    assert np.array_equal(gi, oi)
    assert np.array_equal(gd.view(np.uint32), od.view(np.uint32))


@pytest.mark.parametrize("V,D,k", [(1100, 256, 64), (640, 40, 640), (2000, 100, 1000), (1001, 37, 100), (130, 33, 130)])
def test_large_d_exact(V, D, k):
    cb = li.codebook_clustered(V, D, centres=37, seed=8)
    gi, gd = _gpu(cb, k)
    oi, od = oracle.build_neighbors(cb, k)
    assert np.array_equal(gi, oi)
    assert np.array_equal(gd.view(np.uint32), od.view(np.uint32))


@pytest.mark.parametrize("name,k", [("batch_chain", 1000), ("single_image", 100), ("stress", 1000)])
def test_full_size_sampled_rows(name, k):
    # V = 16384 at the configurations' k: every row is built on the GPU, a seeded sample of
    # rows is recomputed by the oracle one by one; all rows are checked structurally.
    cb = li.config_codebook(name)
    V = cb.shape[0]
    gi, gd = _gpu(cb, k)
    rows = np.random.default_rng(3).choice(V, size=48, replace=False).astype(np.int32)
    oi, od = oracle.build_neighbors(cb, k, rows=rows)
    assert np.array_equal(gi[rows], oi)
    assert np.array_equal(gd[rows].view(np.uint32), od.view(np.uint32))
    assert np.array_equal(gi[:, 0], np.arange(V))
    assert np.all(gd[:, 0] == 0) and np.all(np.diff(gd, axis=1) >= 0)
    assert gi.min() >= 0 and gi.max() < V
    srt = np.sort(gi, axis=1)
    assert np.all(srt[:, 1:] != srt[:, :-1])       # no token twice in a row


def test_argument_errors():
    cb = torch.from_numpy(li.codebook_gaussian(64, 8)).cuda()
    with pytest.raises(lt.LanternError) as e:
        lt.build_neighbors(cb, 65)
    assert e.value.code == -2
    with pytest.raises(lt.LanternError):
        lt.build_neighbors(cb, 0)
    with pytest.raises(ValueError):
        lt.build_neighbors(cb.cpu(), 4)
