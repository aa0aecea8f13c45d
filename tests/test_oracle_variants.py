"""Pins of the oracle's variants: the JSD bound (Section 5.3.2), the cosine neighbour metric
(Section 5.3.1) and the top-k logit filter (Appendix B.2).

  * JSD: the closed form on the collapsed tokens against the definition written out with numpy on
    whole distributions; the prefix rule by brute force; q(x~) = 0 reduces it to a TVD bound of
    delta / ln 2 (the relation behind the matched pairs of Table 3); A under JSD contains A under
    TVD at the same delta; delta >= ln 2 takes the whole neighbourhood;
  * cosine: unit scaling against fp64; the chosen neighbours are the most similar ones under fp64
    cosine similarity; invariance under power-of-two rescaling of single codes (exact in fp32);
  * top-k: the filtered distribution against numpy (ties at the threshold kept); K = 1, K >= V;
    equality with pre-masked logits where the processed logit is the logit itself; the emitted
    token never leaves the target's top-k set; a Monte-Carlo test that plain speculative
    sampling (delta = 0) then reproduces the filtered target distribution.
"""
import dataclasses

import numpy as np
import pytest

import lantern_inputs as li
import oracle


def np_jsd(a, b):
    m = 0.5 * (a + b)
    with np.errstate(divide="ignore", invalid="ignore"):
        ta = np.where(a > 0, a * np.log(a / m), 0.0)
        tb = np.where(b > 0, b * np.log(b / m), 0.0)
    return 0.5 * (ta.sum() + tb.sum())


def collapse(q, A, x):
    qd = q.copy()
    qd[A] = 0.0
    qd[x] = q[A].sum()
    return qd


def rand_q(V, rng, peak=2.0):
    z = rng.normal(size=V) * peak
    e = np.exp(z - z.max())
    return e / e.sum()


# ------------------------------------------------------------------------------------ JSD
def test_jsd_closed_form_against_definition():
    rng = np.random.default_rng(3)
    for _ in range(40):
        V = int(rng.integers(8, 200))
        q = rand_q(V, rng)
        A = rng.choice(V, size=int(rng.integers(1, V)), replace=False)
        x = A[0]
        want = np_jsd(q, collapse(q, A, x))
        got = oracle.jsd_collapsed(q[x], q[A[1:]].sum())
        assert abs(got - want) < 1e-14 + 1e-12 * want
    assert oracle.jsd_collapsed(0.3, 0.0) == 0.0
    assert abs(oracle.jsd_collapsed(0.0, 0.25) - 0.25 * np.log(2)) < 1e-16
    # a zero-mass member changes nothing; the divergence grows with the moved mass
    s = np.linspace(0, 0.9, 50)
    f = np.array([oracle.jsd_collapsed(0.1, t) for t in s])
    assert np.all(np.diff(f) > 0) and f[-1] < np.log(2)


@pytest.mark.parametrize("delta", [0.0, 0.01, 0.1, 0.3, 0.69, 0.7])
def test_jsd_prefix_rule_by_brute_force(delta):
    rng = np.random.default_rng(5)
    V, k = 96, 24
    table = oracle.build_neighbors(li.codebook_gaussian(V, 4, seed=1), k)[0]
    cut = whole = 0
    for t in range(60):
        q = rand_q(V, rng, peak=3.0)
        x = int(rng.integers(V))
        m_want = 0
        for j in range(1, k):
            if np_jsd(q, collapse(q, table[x, : j + 1], x)) < delta:
                m_want = j
            else:
                break
        m, moved, margin = oracle.a_set(q, table[x], delta, oracle.DIV_JSD)
        if margin > 1e-12:
            assert m == m_want
            assert abs(moved - q[table[x, 1 : m + 1]].sum()) < 1e-15
        cut += m < k - 1
        whole += m == k - 1
        # same delta: the JSD of a move never exceeds its TVD, so the JSD set contains the TVD set
        assert m >= oracle.a_set(q, table[x], delta, oracle.DIV_TVD)[0]
    if delta == 0.0:
        assert whole == 0
    if delta >= np.log(2):
        assert cut == 0
    if 0.0 < delta < 0.5:
        assert cut > 0


def test_jsd_with_massless_draft_is_a_tvd_bound():
    rng = np.random.default_rng(8)
    V, k = 128, 40
    table = oracle.build_neighbors(li.codebook_gaussian(V, 4, seed=2), k)[0]
    for delta in (0.2, 0.3):                       # Table 3's TVD settings; matched JSD settings 0.13, 0.2
        for _ in range(30):
            q = rand_q(V, rng)
            x = int(rng.integers(V))
            q[x] = 0.0
            q /= q.sum()
            a = oracle.a_set(q, table[x], delta, oracle.DIV_TVD)
            b = oracle.a_set(q, table[x], delta * np.log(2), oracle.DIV_JSD)
            if min(a[2], b[2]) > 1e-12:
                assert a[:2] == b[:2]
    assert abs(0.3 * np.log(2) - 0.2) < 0.01 and abs(0.2 * np.log(2) - 0.13) < 0.01


def test_verify_under_jsd():
    V, k, N, B = 256, 24, 5, 80
    table = oracle.build_neighbors(li.codebook_gaussian(V, 8, seed=4), k)[0]
    inp = li.verify_inputs(B, N, V, dtype=li.BF16, has_uncond=True, cfg_scale=2.0, sigma_target=1.0,
                           sigma_draft=0.8, rho=0.9, seed=21)
    plain = oracle.verify_inputs(inp, table, 0.0)
    assert np.array_equal(oracle.verify_inputs(inp, table, 0.0, oracle.DIV_JSD).accept_len, plain.accept_len)
    res = oracle.verify_inputs(inp, table, 0.1, oracle.DIV_JSD)
    tv = oracle.verify_inputs(inp, table, 0.1, oracle.DIV_TVD)
    seen = 0
    for b in range(B):
        # first tested node of the root context: q is the unmodified target
        c = 0
        q = oracle.row_distribution(inp.target_logits[0, b, 0], inp.target_logits[1, b, 0], inp.dtype, inp.cfg_scale, inp.T)
        x = inp.draft_tokens[b, c]
        m, moved, _ = oracle.a_set(q, table[x], 0.1, oracle.DIV_JSD)
        assert res.m[b, c] == m and abs(res.qa[b, c] - (q[x] + moved)) < 1e-15
        assert np_jsd(q, collapse(q, table[x, : m + 1], x)) < 0.1 + 1e-12
        assert res.m[b, c] >= tv.m[b, c]
        seen += m > 0
    assert seen > B // 2
    big = oracle.verify_inputs(inp, table, 0.7, oracle.DIV_JSD)      # ln 2 = 0.693: the bound never binds
    t = big.tested.astype(bool)
    assert np.all(big.m[t] == k - 1)
    g = oracle.verify_greedy(inp.target_logits, inp.dtype, inp.cfg_scale, inp.has_uncond, inp.draft_tokens, None,
                             table, 0.1, oracle.DIV_JSD)
    g_tv = oracle.verify_greedy(inp.target_logits, inp.dtype, inp.cfg_scale, inp.has_uncond, inp.draft_tokens, None,
                                table, 0.1)
    assert np.all(g.accept_len >= g_tv.accept_len) and g.accept_len.sum() > g_tv.accept_len.sum()


# ------------------------------------------------------------------------------------ cosine
def test_cosine_neighbours():
    V, D, k = 300, 6, 20
    rng = np.random.default_rng(2)
    cb = (rng.normal(size=(V, D)) * rng.uniform(0.1, 10.0, size=(V, 1))).astype(np.float32)
    unit = oracle.normalize_rows(cb)
    ref = cb.astype(np.float64) / np.linalg.norm(cb.astype(np.float64), axis=1, keepdims=True)
    assert np.abs(unit - ref).max() < 2e-7
    idx, dist = oracle.build_neighbors(cb, k, metric="cosine")
    sim = ref @ ref.T
    for i in range(V):
        assert idx[i, 0] == i
        s = sim[i, idx[i]]
        assert np.all(np.diff(s[1:]) < 1e-6)                       # decreasing similarity
        rest = np.setdiff1d(np.arange(V), idx[i])
        assert s[-1] > sim[i, rest].max() - 1e-6                   # nothing more similar was left out
        assert np.abs(dist[i] - (2.0 - 2.0 * s)).max() < 1e-5
    # cosine ignores the length of a code: power-of-two rescaling is exact in fp32
    scaled = cb * (2.0 ** rng.integers(-6, 7, size=(V, 1))).astype(np.float32)
    assert np.array_equal(oracle.build_neighbors(scaled, k, metric="cosine")[0], idx)
    assert not np.array_equal(oracle.build_neighbors(scaled, k)[0], oracle.build_neighbors(cb, k)[0])
    # a zero code stays zero
    cb0 = cb.copy()
    cb0[7] = 0.0
    assert not oracle.normalize_rows(cb0)[7].any()


# ------------------------------------------------------------------------------------ top-k
def np_topk_softmax(z, K):
    z = np.asarray(z, dtype=np.float64).copy()
    if 0 < K < z.size:
        kth = np.sort(z)[::-1][K - 1]
        z[z < kth] = -np.inf
    e = np.exp(z - z.max())
    return e / e.sum()


@pytest.mark.parametrize("K", [1, 3, 50, 127, 128, 1000, 0])
def test_top_k_distribution(K):
    V = 128
    rng = np.random.default_rng(11)
    for dtype in (li.F32, li.BF16):
        inp = li.verify_inputs(6, 0, V, dtype=dtype, has_uncond=False, cfg_scale=1.0, sigma_target=2.0,
                               sigma_draft=1.0, rho=0.0, seed=int(rng.integers(1000)))
        for b in range(6):
            row = inp.target_logits[0, b, 0]
            z = row.astype(np.float64) if dtype == li.F32 else (row.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
            got = oracle.row_distribution(row, None, dtype, 1.0, 1.0, top_k=K)
            want = np_topk_softmax(z, K)
            assert np.abs(got - want).max() < 1e-15
            kept = int((got > 0).sum())
            if 0 < K < V:
                assert kept >= K                                    # ties at the threshold are all kept
                if dtype == li.F32:
                    assert kept == K
            else:
                assert kept == V


def test_top_k_ties_are_kept():
    z = np.array([1.0, 3.0, 2.0, 2.0, 2.0, 0.5, -1.0, 0.0], dtype=np.float32)
    q = oracle.row_distribution(z, None, li.F32, 1.0, 1.0, top_k=2)
    assert (q > 0).tolist() == [False, True, True, True, True, False, False, False]
    assert abs(q[1] - np.e / (np.e + 3)) < 1e-15


def test_top_k_equals_premasked_logits():
    V, k, N, B, K = 128, 12, 4, 60, 20
    table = oracle.build_neighbors(li.codebook_gaussian(V, 4, seed=6), k)[0]
    inp = li.verify_inputs(B, N, V, dtype=li.F32, has_uncond=False, cfg_scale=1.0, sigma_target=1.5,
                           sigma_draft=1.5, rho=0.0, seed=33)

    def mask(a):
        a = a.copy()
        flat = a.reshape(-1, V)
        for r in flat:
            kth = np.sort(r)[::-1][K - 1]
            r[r < kth] = -np.inf
        return a

    masked = dataclasses.replace(inp, target_logits=mask(inp.target_logits), draft_logits=mask(inp.draft_logits))
    for div in (oracle.DIV_TVD, oracle.DIV_JSD):
        a = oracle.verify_inputs(inp, table, 0.2, div, top_k=K)
        b = oracle.verify_inputs(masked, table, 0.2, div)
        for f in ("accept_len", "next_token", "accept_path", "status", "qa", "px", "m"):
            assert np.array_equal(getattr(a, f), getattr(b, f)), f
        assert a.accept_len.sum() > 0
    # the emitted token lies in the target's top-k set of the context where the walk stopped
    a = oracle.verify_inputs(inp, table, 0.2, top_k=K)
    for b in range(B):
        prev = a.accept_path[b, a.accept_len[b] - 1] if a.accept_len[b] else -1
        q = oracle.row_distribution(inp.target_logits[0, b, prev + 1], None, li.F32, 1.0, 1.0, top_k=K)
        assert q[a.next_token[b]] > 0


def test_top_k_plain_speculative_sampling_keeps_the_filtered_target():
    """delta = 0, one draft: the emitted first token (accepted draft or resample) follows the top-k target."""
    V, K, trials = 12, 5, 40000
    rng = np.random.default_rng(17)
    tl = rng.normal(size=V).astype(np.float32) * 1.5
    dl = rng.normal(size=V).astype(np.float32) * 1.5
    q = np_topk_softmax(tl, K)
    p = np_topk_softmax(dl, K)
    tokens = rng.choice(V, size=trials, p=p).astype(np.int32).reshape(trials, 1)
    target = np.broadcast_to(tl, (1, trials, 2, V)).copy()
    draft = np.broadcast_to(dl, (trials, 2, V)).copy()
    uni = rng.random((trials, 2)).astype(np.float32)
    table = np.arange(V, dtype=np.int32)[:, None]
    res = oracle.verify(target, draft, li.F32, 1.0, 0, 1.0, tokens, None, table, 0.0, uni, top_k=K)
    first = np.where(res.accept_len > 0, tokens[:, 0], res.next_token)
    counts = np.bincount(first, minlength=V)
    assert counts[q == 0].sum() == 0
    keep = q > 0
    chi2 = ((counts[keep] - trials * q[keep]) ** 2 / (trials * q[keep])).sum()
    assert chi2 < 30.0          # 4 degrees of freedom (5 kept tokens): P(chi2 > 30) < 1e-5


# ------------------------------------------------------------------------------------ all-token aggregation
def test_aggregate_all():
    """agg[x] = sum_{A_{k,delta}(x)} q: delta >= 1 is a product with B_k's 0/1 matrix, delta = 0 and k = 1
    give q itself, and every entry equals a numpy prefix sum cut at the bound."""
    V, k, rows = 200, 12, 5
    table = oracle.build_neighbors(li.codebook_gaussian(V, 4, seed=9), k)[0]
    inp = li.verify_inputs(rows, 0, V, dtype=li.BF16, has_uncond=True, cfg_scale=2.0, sigma_target=1.0,
                           sigma_draft=1.0, rho=0.5, seed=4)
    rc, ru = inp.target_logits[0, :, 0], inp.target_logits[1, :, 0]
    q = np.stack([oracle.row_distribution(rc[r], ru[r], li.BF16, 2.0, 1.0) for r in range(rows)])
    adj = np.zeros((V, V))
    adj[np.arange(V)[:, None], table] = 1.0
    agg, m, _ = oracle.aggregate_all(rc, ru, li.BF16, 2.0, 1.0, table, 1.5)
    assert np.abs(agg - q @ adj.T).max() < 1e-14 and np.all(m == k - 1)
    agg0, m0, _ = oracle.aggregate_all(rc, ru, li.BF16, 2.0, 1.0, table, 0.0)
    assert np.array_equal(agg0, q) and not m0.any()
    agg1, _, _ = oracle.aggregate_all(rc, ru, li.BF16, 2.0, 1.0, table[:, :1], 0.3)
    assert np.array_equal(agg1, q)
    delta = 0.05
    agg, m, margin = oracle.aggregate_all(rc, ru, li.BF16, 2.0, 1.0, table, delta)
    cut = 0
    for r in range(rows):
        for x in range(V):
            cs = np.cumsum(q[r, table[x, 1:]])
            fits = cs < np.float32(delta)
            want = k - 1 if fits.all() else int(np.argmin(fits))
            if margin[r, x] > 1e-12:
                assert m[r, x] == want
                assert abs(agg[r, x] - (q[r, x] + (cs[want - 1] if want else 0.0))) < 1e-15
            cut += want < k - 1
    assert cut > rows * V // 10
    assert np.all(oracle.aggregate_all(rc, ru, li.BF16, 2.0, 1.0, table, 0.2)[0] >= agg - 1e-15)
