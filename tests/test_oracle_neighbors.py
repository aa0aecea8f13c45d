"""Pins of the oracle's neighbour-table builder (Algorithm 2, "Precompute B_k" block).

None of these re-types the oracle's loop: they compare it with numpy's own sort on exactly
representable distances, with scipy's k-d tree, with the cosine order on unit-norm codebooks,
and with structural facts the paper states (x~ is always in B_k(x~); increasing distance).
"""
import numpy as np
import pytest
from scipy.spatial import cKDTree

import lantern_inputs as li
import oracle


def test_integer_codebook_matches_numpy_stable_sort():
    # integer entries: every squared distance is an exact small integer in fp32 and fp64, so
    # the (distance, index) order is unambiguous and numpy's stable argsort is the definition.
    cb = li.codebook_integer(96, 5, seed=7)
    V = cb.shape[0]
    k = 17
    idx, dist = oracle.build_neighbors(cb, k)
    d2 = ((cb[:, None, :].astype(np.float64) - cb[None, :, :].astype(np.float64)) ** 2).sum(-1)
    for i in range(V):
        others = np.array([j for j in range(V) if j != i])
        order = others[np.argsort(d2[i, others], kind="stable")]
        want = np.concatenate([[i], order[: k - 1]])
        assert np.array_equal(idx[i], want), i
        assert np.array_equal(dist[i].astype(np.float64), d2[i, want])


def test_self_first_even_with_duplicate_codes():
    cb = li.codebook_integer(40, 3, seed=3)
    cb[25] = cb[4]  # an exact duplicate with a smaller index
    cb[31] = cb[4]
    idx, dist = oracle.build_neighbors(cb, 5)
    assert np.array_equal(idx[:, 0], np.arange(40))          # x~ in B_k(x~), slot 0
    assert np.all(dist[:, 0] == 0.0)
    assert list(idx[25, :3]) == [25, 4, 31]                   # ties by smaller index after self
    assert list(idx[31, :3]) == [31, 4, 25]
    assert list(idx[4, :3]) == [4, 25, 31]


@pytest.mark.parametrize("V,D,k", [(257, 8, 32), (512, 3, 512), (64, 1, 7)])
def test_structure(V, D, k):
    cb = li.codebook_gaussian(V, D, seed=11, normalise=(D > 1))
    idx, dist = oracle.build_neighbors(cb, k)
    assert idx.shape == (V, k) and dist.shape == (V, k)
    assert np.array_equal(idx[:, 0], np.arange(V))
    assert np.all(dist[:, 0] == 0.0)
    assert np.all(np.diff(dist, axis=1) >= 0.0)               # increasing distance order
    assert idx.min() >= 0 and idx.max() < V
    for i in range(V):
        assert len(set(idx[i].tolist())) == k                 # a set: no repeated token
    if k == V:
        assert np.array_equal(np.sort(idx, axis=1), np.tile(np.arange(V), (V, 1)))


def test_against_kdtree_and_double_precision():
    cb = li.codebook_gaussian(700, 8, seed=5)
    k = 40
    idx, dist = oracle.build_neighbors(cb, k)
    tree = cKDTree(cb.astype(np.float64))
    dd, ii = tree.query(cb.astype(np.float64), k=k)
    # same neighbour *sets* wherever the k-th and (k+1)-th distances are not within rounding
    d_next = tree.query(cb.astype(np.float64), k=k + 1)[0][:, -1]
    clear = (d_next ** 2 - dd[:, -1] ** 2) > 1e-5
    assert clear.mean() > 0.9
    for i in np.nonzero(clear)[0]:
        assert set(idx[i].tolist()) == set(ii[i].tolist())
    # stored distances are the squared l2 distances, to fp32 accuracy
    exact = ((cb[:, None, :].astype(np.float64) - cb[idx].astype(np.float64)) ** 2).sum(-1)
    np.testing.assert_allclose(dist, exact, rtol=2e-6, atol=1e-7)
    # the double-precision order differs from the fp32 order in few rows, if any
    assert oracle.count_order_differences(cb, idx) <= 0.05 * cb.shape[0]


def test_cosine_order_on_unit_norm_codebook():
    # Section 5.3.1 / Table 3: l2 and cosine proximity behave alike; on unit-norm codes they
    # are the same order because ||a-b||^2 = 2 - 2 cos(a,b).
    cb = li.codebook_gaussian(400, 8, seed=9, normalise=True)
    k = 25
    idx, dist = oracle.build_neighbors(cb, k)
    c = cb.astype(np.float64)
    c /= np.linalg.norm(c, axis=1, keepdims=True)
    cos = c @ c.T
    for i in range(400):
        got = cos[i, idx[i, 1:]]
        assert np.all(np.diff(got) <= 2e-6)                   # descending cosine, up to fp32 ties
        kth = np.sort(np.delete(cos[i], i))[::-1][k - 2]
        assert got.min() >= kth - 2e-6


def test_bad_arguments():
    cb = li.codebook_gaussian(16, 4, seed=1)
    with pytest.raises(ValueError):
        oracle.build_neighbors(cb, 17)
    with pytest.raises(ValueError):
        oracle.build_neighbors(cb, 0)
    cb[3, 1] = np.nan
    with pytest.raises(ValueError):
        oracle.build_neighbors(cb, 4)
