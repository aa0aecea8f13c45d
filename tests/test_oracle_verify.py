"""Pins of the oracle's verification step against what the paper and the mathematics fix.

  * k = 1 or delta = 0 is standard speculative sampling (Section 2): identical outputs to a
    separately written textbook sampler, and a Monte-Carlo chi-square of the emitted token
    against the target q;
  * D_TV(q_{k,delta}, q) < delta and equals the moved mass, by brute force (Section 4.3);
  * maximality of the prefix (Algorithm 2, second block);
  * relaxed acceptance >= original, monotone in k and delta (eq. 1, Table 1's trend);
  * residual support and normalisation (Section 4.3);
  * large delta gives B_k and eq. 1;
  * the uniform-distribution closed form, exact in binary floating point;
  * the exact emitted-token law for delta > 0 on a tiny vocabulary (Monte-Carlo chi-square);
  * branching trees at delta = 0 stay lossless (multi-round rejection);
  * a hand-worked example kept under tests/golden/.
"""
import json
import os

import numpy as np
import pytest
from scipy import stats

import lantern_inputs as li
import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


# ---------------------------------------------------------------------------------------
# helpers written independently of the oracle
# ---------------------------------------------------------------------------------------
def np_softmax(z):
    z = np.asarray(z, dtype=np.float64)
    e = np.exp(z - z.max())
    return e / e.sum()


def textbook_chain(q_rows, p_rows, tokens, uniforms):
    """Leviathan et al. speculative sampling on a chain (Section 2 of the paper)."""
    N = len(tokens)
    for t in range(N):
        q, p = q_rows[t], p_rows[t]
        x = tokens[t]
        if uniforms[t] < min(1.0, q[x] / p[x]) if p[x] > 0 else True:
            continue
        res = np.maximum(q - p, 0.0)
        cdf = np.cumsum(res)
        tok = int(np.searchsorted(cdf, uniforms[N] * cdf[-1], side="right"))
        return t, min(tok, len(q) - 1)
    cdf = np.cumsum(q_rows[N])
    return N, int(np.searchsorted(cdf, uniforms[N] * cdf[-1], side="right"))


def small_case(B, N, V, seed, parents=None, dtype=li.F32, has_uncond=False, **kw):
    return li.verify_inputs(B, N, V, dtype=dtype, has_uncond=has_uncond, cfg_scale=kw.pop("cfg_scale", 1.0),
                            sigma_target=kw.pop("sigma_target", 1.5), sigma_draft=kw.pop("sigma_draft", 0.5),
                            parents=parents, seed=seed, **kw)


def identity_table(V):
    return np.arange(V, dtype=np.int32)[:, None]


# ---------------------------------------------------------------------------------------
# P1: reduction to standard speculative sampling
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("mode", ["k1", "delta0"])
def test_reduces_to_textbook_sampler(mode):
    V, N, B = 64, 5, 200
    inp = small_case(B, N, V, seed=101)
    if mode == "k1":
        table, delta = identity_table(V), 0.3
    else:
        table, delta = oracle.build_neighbors(li.codebook_gaussian(V, 4, seed=2), 9)[0], 0.0
    res = oracle.verify_inputs(inp, table, delta)
    n_rejected = 0
    for b in range(B):
        q_rows = [np_softmax(inp.target_logits[0, b, t]) for t in range(N + 1)]
        p_rows = [np_softmax(inp.draft_logits[b, t]) for t in range(N + 1)]
        al, tok = textbook_chain(q_rows, p_rows, inp.draft_tokens[b], inp.uniforms[b].astype(np.float64))
        assert res.accept_len[b] == al
        assert res.next_token[b] == tok
        n_rejected += al < N
    assert 0 < n_rejected < B  # both branches exercised
    assert np.all(res.status == 0)


def test_k1_monte_carlo_is_lossless():
    # emitted first token ~ q when x~ ~ p, and acceptance rate = sum min(p, q) = 1 - TV(p, q)
    V, B = 8, 400_000
    rng = np.random.default_rng(77)
    lq = rng.normal(0, 1.2, V).astype(np.float32)
    lp = (lq + rng.normal(0, 0.8, V)).astype(np.float32)
    q, p = np_softmax(lq), np_softmax(lp)
    tokens = rng.choice(V, size=(B, 1), p=p).astype(np.int32)
    target = np.broadcast_to(lq, (1, B, 2, V)).copy()
    draft = np.broadcast_to(lp, (B, 2, V)).copy()
    un = rng.random((B, 2), dtype=np.float32)
    res = oracle.verify(target, draft, li.F32, 1.0, 0, 1.0, tokens, None, identity_table(V), 0.25, un)
    emitted = np.where(res.accept_len == 1, tokens[:, 0], res.next_token)
    counts = np.bincount(emitted, minlength=V)
    chi = stats.chisquare(counts, q * B)
    assert chi.pvalue > 1e-4, chi
    rate = (res.accept_len == 1).mean()
    assert abs(rate - np.minimum(p, q).sum()) < 5 * np.sqrt(0.25 / B)
    # after an accepted draft the bonus token is a plain draw from q (Algorithm 1, last line)
    acc = res.accept_len == 1
    chi2 = stats.chisquare(np.bincount(res.next_token[acc], minlength=V), q * acc.sum())
    assert chi2.pvalue > 1e-4, chi2


# ---------------------------------------------------------------------------------------
# P2, P3, P6, P7, P8 on a mid-size vocabulary with a real neighbour table
# ---------------------------------------------------------------------------------------
@pytest.fixture(scope="module")
def mid():
    V, k = 512, 48
    table = oracle.build_neighbors(li.codebook_gaussian(V, 8, seed=4), k)[0]
    inp = small_case(40, 6, V, seed=202, dtype=li.BF16, has_uncond=True, cfg_scale=3.0, sigma_target=1.0,
                     sigma_draft=1.5, rho=0.9)
    return V, k, table, inp


def _rows(inp, b, t):
    tq = inp.target_logits
    q = oracle.row_distribution(tq[0, b, t], tq[1, b, t] if inp.has_uncond else None, inp.dtype, inp.cfg_scale, inp.T)
    p = oracle.row_distribution(inp.draft_logits[b, t], None, inp.dtype, 1.0, inp.T)
    return q, p


@pytest.mark.parametrize("delta", [0.05, 0.2, 0.4])
def test_tvd_bound_and_maximality(mid, delta):
    V, k, table, inp = mid
    res = oracle.verify_inputs(inp, table, delta)
    seen = 0
    for b in range(inp.B):
        for t in range(inp.N):
            if not res.tested[b, t]:
                continue
            seen += 1
            q, p = _rows(inp, b, t)       # chain: node t is tested in context row t, first sibling
            x = inp.draft_tokens[b, t]
            m = res.m[b, t]
            A = table[x, : m + 1]
            qd = q.copy()
            qd[A] = 0.0
            qd[x] = q[A].sum()            # q_{k,delta}(.|D=x~) of Section 4.3
            tv = 0.5 * np.abs(qd - q).sum()
            d32 = float(np.float32(delta))
            assert tv < d32
            assert abs(tv - (res.qa[b, t] - q[x])) < 1e-12          # TVD equals the moved mass
            assert abs(res.qa[b, t] - q[A].sum()) < 1e-12
            assert abs(res.px[b, t] - p[x]) < 1e-12
            if m < k - 1:                                            # maximal prefix
                assert tv + q[table[x, m + 1]] >= d32
    assert seen > inp.B


def test_relaxed_accept_dominates_and_is_monotone(mid):
    V, k, table, inp = mid
    base = oracle.verify_inputs(inp, identity_table(V), 0.0)
    prev = None
    for kk in (1, 8, 48):
        for delta in (0.0, 0.05, 0.2, 0.4, 2.0):
            res = oracle.verify_inputs(inp, np.ascontiguousarray(table[:, :kk]), delta)
            # compare on first-position nodes (always tested, same context for every setting)
            qa = res.qa[:, 0]
            assert np.all(qa >= base.qa[:, 0] - 1e-15)              # eq. 1 remark: never below original
            if delta > 0 and kk == 48:
                assert np.all(qa >= prev - 1e-15)                   # non-decreasing in delta
            prev = qa if kk == 48 else None
    # non-decreasing in k at fixed delta
    qa_k = [oracle.verify_inputs(inp, np.ascontiguousarray(table[:, :kk]), 0.3).qa[:, 0] for kk in (1, 4, 16, 48)]
    for a, b_ in zip(qa_k, qa_k[1:]):
        assert np.all(b_ >= a - 1e-15)


def test_large_delta_gives_full_neighbourhood(mid):
    V, k, table, inp = mid
    res = oracle.verify_inputs(inp, table, 1.5)
    for b in range(inp.B):
        q, p = _rows(inp, b, 0)
        x = inp.draft_tokens[b, 0]
        assert res.m[b, 0] == k - 1
        assert abs(res.qa[b, 0] - q[table[x]].sum()) < 1e-12         # eq. 1 numerator over B_k
        assert (res.accept_len[b] >= 1) == (inp.uniforms[b, 0] * p[x] < q[table[x]].sum())


def test_residual_support_and_draw(mid):
    V, k, table, inp = mid
    delta = 0.05
    res = oracle.verify_inputs(inp, table, delta)
    checked = 0
    for b in range(inp.B):
        t = res.accept_len[b]
        if t == inp.N:
            continue
        q, p = _rows(inp, b, t)
        x = inp.draft_tokens[b, t]
        A = table[x, : res.m[b, t] + 1]
        qd = q.copy()
        qd[A] = 0.0
        qd[x] = q[A].sum()
        w = np.maximum(qd - p, 0.0)
        assert np.all(w[A] == 0.0)                                   # no mass left inside A (x~ included)
        assert abs(w.sum() - res.w[b]) < 1e-12
        assert w.sum() >= p[x] - qd[x] - 1e-12                       # positive total weight after a rejection
        tok = res.next_token[b]
        assert w[tok] > 0 and tok not in set(A.tolist())
        cdf = np.cumsum(w)
        assert tok == int(np.searchsorted(cdf, np.float64(inp.uniforms[b, inp.N]) * cdf[-1], side="right"))
        checked += 1
    assert checked > 5


# ---------------------------------------------------------------------------------------
# P12: uniform distributions, exact in binary floating point
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("V,k,delta,m_want", [(16, 12, 0.25, 3), (16, 3, 0.25, 2), (64, 64, 0.5, 31),
                                                (64, 64, 0.0, 0), (16, 12, 0.26, 4), (16, 16, 1.0, 15)])
def test_uniform_closed_form(V, k, delta, m_want):
    # all logits equal: q = 1/V exactly, prefix sums j/V are exact, so the strict bound
    # s_j < delta keeps j <= ceil(delta V) - 1 neighbours (capped at k - 1).
    table = oracle.build_neighbors(li.codebook_gaussian(V, 4, seed=8), k)[0]
    target = np.zeros((1, 3, 2, V), np.float32)
    draft = np.zeros((3, 2, V), np.float32)
    tokens = np.array([[0], [5], [V - 1]], np.int32)
    un = np.full((3, 2), 0.5, np.float32)
    res = oracle.verify(target, draft, li.F32, 1.0, 0, 1.0, tokens, None, table, delta, un)
    assert m_want == min(k - 1, int(np.ceil(np.float32(delta) * V)) - 1 if delta > 0 else 0)
    assert np.all(res.m[:, 0] == m_want)
    assert np.all(res.qa[:, 0] == (1 + m_want) / V)
    assert np.all(res.accept_len == 1)


# ---------------------------------------------------------------------------------------
# P11: exact emitted-token law with delta > 0
# ---------------------------------------------------------------------------------------
def test_relaxed_emitted_token_law():
    V, k, delta, B = 8, 4, 0.3, 400_000
    rng = np.random.default_rng(5)
    lq = rng.normal(0, 1.0, V).astype(np.float32)
    lp = (lq + rng.normal(0, 1.0, V)).astype(np.float32)
    q, p = np_softmax(lq), np_softmax(lp)
    table = oracle.build_neighbors(li.codebook_gaussian(V, 2, seed=6, normalise=False), k)[0]
    # law of the first emitted token: sum_x~ p(x~) [ a(x~) 1{y = x~} + (1 - a(x~)) w_x~(y) / W_x~ ]
    law = np.zeros(V)
    n_relaxed = 0
    for x in range(V):
        s, A = 0.0, [x]
        for n in table[x, 1:]:
            if s + q[n] < np.float32(delta):
                s += q[n]
                A.append(n)
            else:
                break
        n_relaxed += len(A) > 1
        qd = q.copy()
        qd[A] = 0.0
        qd[x] = q[x] + s
        a = min(1.0, qd[x] / p[x])
        w = np.maximum(qd - p, 0.0)
        law[x] += p[x] * a
        if a < 1.0:
            law += p[x] * (1.0 - a) * w / w.sum()
    assert n_relaxed >= 3 and abs(law.sum() - 1.0) < 1e-12
    assert np.abs(law - q).max() > 0.01  # the relaxed law really differs from q here
    tokens = rng.choice(V, size=(B, 1), p=p).astype(np.int32)
    target = np.broadcast_to(lq, (1, B, 2, V)).copy()
    draft = np.broadcast_to(lp, (B, 2, V)).copy()
    un = rng.random((B, 2), dtype=np.float32)
    res = oracle.verify(target, draft, li.F32, 1.0, 0, 1.0, tokens, None, table, delta, un)
    emitted = np.where(res.accept_len == 1, tokens[:, 0], res.next_token)
    chi = stats.chisquare(np.bincount(emitted, minlength=V), law * B)
    assert chi.pvalue > 1e-4, chi
    # and it is NOT q: the same statistic against q must fail decisively
    assert stats.chisquare(np.bincount(emitted, minlength=V), q * B).pvalue < 1e-6


# ---------------------------------------------------------------------------------------
# P9, P10: trees
# ---------------------------------------------------------------------------------------
def test_chain_as_tree_is_identical(mid):
    V, k, table, inp = mid
    a = oracle.verify_inputs(inp, table, 0.3)
    inp2 = li.VerifyInputs(**{**inp.__dict__, "tree_parents": li.chain_parents(inp.B, inp.N)})
    b = oracle.verify_inputs(inp2, table, 0.3)
    for f in ("accept_len", "next_token", "accept_path", "status", "tested", "qa", "px", "m"):
        assert np.array_equal(getattr(a, f), getattr(b, f)), f


def test_branching_tree_delta0_is_lossless():
    # root with three children drawn without replacement from p; multi-round rejection must
    # emit a first token distributed exactly as q (the base tree method is distribution-
    # preserving, Section 5.1).
    V, B, C = 8, 300_000, 3
    rng = np.random.default_rng(123)
    lq = rng.normal(0, 1.2, V).astype(np.float32)
    lp = (lq + rng.normal(0, 1.0, V)).astype(np.float32)
    q = np_softmax(lq)
    gumbel = -np.log(-np.log(rng.random((B, V))))
    tokens = np.argsort(-(lp.astype(np.float64) + gumbel), axis=1)[:, :C].astype(np.int32)
    parents = np.full((B, C), -1, np.int32)
    target = np.broadcast_to(lq, (1, B, C + 1, V)).copy()
    draft = np.broadcast_to(lp, (B, C + 1, V)).copy()
    un = rng.random((B, C + 1), dtype=np.float32)
    table = oracle.build_neighbors(li.codebook_gaussian(V, 2, seed=6, normalise=False), 4)[0]
    res = oracle.verify(target, draft, li.F32, 1.0, 0, 1.0, tokens, parents, table, 0.0, un)
    first = np.where(res.accept_len >= 1, tokens[np.arange(B), np.maximum(res.accept_path[:, 0], 0)], res.next_token)
    chi = stats.chisquare(np.bincount(first, minlength=V), q * B)
    assert chi.pvalue > 1e-4, chi
    # siblings matter: some sequences accept the 2nd or 3rd child
    assert (res.accept_path[:, 0] >= 1).mean() > 0.02
    # more children accept more often than a single draft would
    assert (res.accept_len >= 1).mean() > np.minimum(np_softmax(lp), q).sum() + 0.02


def test_tree_walk_follows_parents():
    V, k = 256, 16
    table = oracle.build_neighbors(li.codebook_gaussian(V, 8, seed=4), k)[0]
    par = li.tree_parents(30, 20, depth=4, seed=9)
    inp = small_case(30, 20, V, seed=303, parents=par, dtype=li.BF16, has_uncond=True, cfg_scale=2.0,
                     sigma_target=1.0, sigma_draft=0.4, rho=0.95)
    res = oracle.verify_inputs(inp, table, 0.4)
    assert res.accept_len.max() >= 2
    for b in range(30):
        prev = -1
        for d in range(res.accept_len[b]):
            node = res.accept_path[b, d]
            assert par[b, node] == prev and res.tested[b, node]
            prev = node
        assert np.all(res.accept_path[b, res.accept_len[b]:] == -1)
        # every tested node hangs off the accepted path
        for node in np.nonzero(res.tested[b])[0]:
            assert par[b, node] in [-1] + res.accept_path[b, : res.accept_len[b]].tolist()


# ---------------------------------------------------------------------------------------
# hand-worked example
# ---------------------------------------------------------------------------------------
def test_hand_worked_example():
    g = json.load(open(os.path.join(HERE, "golden", "hand_example_v4.json")))
    V = g["V"]
    table = np.array(g["neighbors"], np.int32)
    lq = np.log(np.array(g["q"])).astype(np.float32)
    lp = np.log(np.array(g["p"])).astype(np.float32)
    for case in g["cases"]:
        N = len(case["tokens"])
        if "q" in case:
            lq = np.log(np.array(case["q"])).astype(np.float32)
            lp = np.log(np.array(case["p"])).astype(np.float32)
        target = np.broadcast_to(lq, (1, 1, N + 1, V)).copy()
        draft = np.broadcast_to(lp, (1, N + 1, V)).copy()
        res = oracle.verify(target, draft, li.F32, 1.0, 0, 1.0, np.array([case["tokens"]], np.int32),
                            np.array([case["parents"]], np.int32), table, case["delta"],
                            np.array([case["uniforms"]], np.float32))
        assert res.accept_len[0] == case["accept_len"], case["_why"]
        assert res.next_token[0] == case["next_token"], case["_why"]
        tested = res.tested[0].astype(bool)
        np.testing.assert_allclose(res.qa[0][tested], np.array(case["qa"])[tested], rtol=1e-6)
        np.testing.assert_allclose(res.px[0][tested], np.array(case["px"])[tested], rtol=1e-6)
        assert list(res.m[0][tested]) == list(np.array(case["m"])[tested])
        np.testing.assert_allclose(res.w[0], case["W"], rtol=1e-6, atol=1e-12)
        if "accept_path" in case:
            assert list(res.accept_path[0]) == case["accept_path"]


# ---------------------------------------------------------------------------------------
# guidance and temperature (Appendix B.2 gives the scales; the combine is the usual
# classifier-free-guidance form in logit space)
# ---------------------------------------------------------------------------------------
def test_guidance_and_temperature_form():
    rng = np.random.default_rng(3)
    V = 200
    c = li.bf16_bits_to_f32(li.f32_to_bf16_bits(rng.normal(0, 1, V).astype(np.float32)))
    u = li.bf16_bits_to_f32(li.f32_to_bf16_bits(rng.normal(0, 1, V).astype(np.float32)))
    cb, ub = li.f32_to_bf16_bits(c), li.f32_to_bf16_bits(u)
    for s, T in [(7.5, 1.0), (4.0, 0.7), (3.0, 2.0)]:
        got = oracle.row_distribution(cb, ub, li.BF16, s, T)
        want = np_softmax((u.astype(np.float64) + s * (c.astype(np.float64) - u.astype(np.float64))) / T)
        np.testing.assert_allclose(got, want, rtol=2e-5)
        assert abs(got.sum() - 1.0) < 1e-12
    # scale 1 is the conditional branch alone, scale 0 the unconditional branch alone
    np.testing.assert_allclose(oracle.row_distribution(cb, ub, li.BF16, 1.0, 1.0), np_softmax(c), rtol=1e-6)
    np.testing.assert_allclose(oracle.row_distribution(cb, ub, li.BF16, 0.0, 1.0), np_softmax(u), rtol=1e-6)
    # no unconditional branch: plain tempered softmax, on fp32 storage too
    np.testing.assert_allclose(oracle.row_distribution(c, None, li.F32, 9.0, 0.5), np_softmax(c / 0.5), rtol=1e-6)
    # T -> small sharpens towards the arg max
    assert oracle.row_distribution(c, None, li.F32, 1.0, 0.05).argmax() == c.argmax()


# ---------------------------------------------------------------------------------------
# data faults are reported, never fatal
# ---------------------------------------------------------------------------------------
def test_status_bits():
    V, k = 64, 8
    table = oracle.build_neighbors(li.codebook_gaussian(V, 4, seed=4), k)[0]
    inp = small_case(6, 3, V, seed=9)
    inp.draft_tokens[1, 1] = V
    inp.uniforms[2, 0] = 1.0
    inp.target_logits[0, 3, 0, 5] = np.nan
    inp.target_logits[0, 4, 0, :] = -np.inf
    inp.target_logits[0, 5, 0, 7] = -np.inf           # a masked token is legal
    par = li.chain_parents(6, 3)
    par[0, 2] = 2
    inp.tree_parents = par
    res = oracle.verify_inputs(inp, table, 0.2)
    assert res.status[0] == oracle.ST_BAD_PARENT and res.next_token[0] == -1 and res.accept_len[0] == 0
    assert res.status[1] == oracle.ST_BAD_TOKEN
    assert res.status[2] == oracle.ST_BAD_UNIFORM
    assert res.status[3] == oracle.ST_NONFINITE and res.next_token[3] == -1
    assert res.status[4] == oracle.ST_NONFINITE
    assert res.status[5] == 0 and res.next_token[5] >= 0
    bad = table.copy()
    bad[:, 1] = V + 3
    res = oracle.verify_inputs(small_case(2, 2, V, seed=10), bad, 0.2)
    assert np.all(res.status & oracle.ST_BAD_TABLE)


# ---------------------------------------------------------------------------------------
# a residual without weight (reading R10): reported, next token from the context's own target
# ---------------------------------------------------------------------------------------
def test_residual_without_weight_draws_from_the_target():
    V, k = 16, 3
    table = oracle.build_neighbors(li.codebook_gaussian(V, 3, seed=4), k)[0]
    inp = small_case(6, 2, V, seed=301)
    inp.draft_logits[:] = inp.target_logits[0]          # drafter = target
    for b in (0, 1, 2):
        x = int(inp.draft_tokens[b, 0])
        inp.target_logits[0, b, 0, table[x]] = -np.inf  # the drafted token and its neighbours carry no mass
        inp.draft_logits[b, 0, table[x]] = -np.inf
    res = oracle.verify_inputs(inp, table, 0.4)
    for b in (0, 1, 2):
        q = np_softmax(inp.target_logits[0, b, 0])
        cdf = np.cumsum(q)
        want = int(np.searchsorted(cdf, np.float64(inp.uniforms[b, 2]) * cdf[-1], side="right"))
        assert res.status[b] == oracle.ST_DEGENERATE and res.accept_len[b] == 0 and res.w[b] == 0.0
        assert res.next_token[b] == want and q[want] > 0
    # drafter = target elsewhere: the ratio is 1 and every draft is accepted
    assert (res.status[3:] == 0).all() and (res.accept_len[3:] == 2).all()


def test_degenerate_threshold_is_a_threshold():
    """W just above / below the threshold: p differs from q on two tokens by +-e, so the residual weighs e."""
    V = 8
    table = identity_table(V)
    for e, degenerate in [(3e-5, False), (3e-6, True)]:
        q = np.full(V, 1.0 / V)
        p = q.copy()
        p[0] += e          # the drafted token: p > q, so it can be rejected
        p[1] -= e
        inp = small_case(1, 1, V, seed=1)
        inp.target_logits[0, 0, 0] = np.log(q).astype(np.float32)
        inp.draft_logits[0, 0] = np.log(p).astype(np.float32)
        inp.draft_tokens[0, 0] = 0
        inp.uniforms[0] = [0.9999999, 0.5]
        res = oracle.verify_inputs(inp, table, 0.0)
        assert res.accept_len[0] == 0
        assert bool(res.status[0] & oracle.ST_DEGENERATE) == degenerate, (e, res.w[0])
        assert abs(res.w[0] - e) < 0.2 * e
        if not degenerate:
            assert res.next_token[0] == 1              # the only token with residual weight
    # the threshold is an argument: at 0 only an exactly empty residual counts
    assert not oracle.verify_inputs(inp, table, 0.0, degenerate_eps=0.0).status[0]


# ---------------------------------------------------------------------------------------
# qa_mag (the magnitude the GPU comparison divides the error of sum_A q by) against a numpy replay
# ---------------------------------------------------------------------------------------
def test_qa_magnitude_matches_a_numpy_replay_of_the_sibling_rounds():
    """For the first child of a context the magnitude is sum_A q itself.  After a rejection the next target is
    (q' - p') / W on the surviving tokens, evaluated from terms of size q' and p': the magnitude carried
    forward is (mag + p') / W there and 0 elsewhere.  Replayed here with numpy on a 3-children root."""
    V, k, delta = 12, 4, 0.15
    table = oracle.build_neighbors(li.codebook_gaussian(V, 3, seed=9), k)[0]
    parents = np.array([[-1, -1, -1]], dtype=np.int32)
    checked = 0
    for seed in range(40):
        inp = small_case(1, 3, V, seed=400 + seed, parents=parents, sigma_draft=1.5)
        inp.uniforms[0, :3] = 0.999          # reject whenever the rule allows it: sibling rounds happen
        res = oracle.verify_inputs(inp, table, delta)
        q = np_softmax(inp.target_logits[0, 0, 0])
        p = np_softmax(inp.draft_logits[0, 0])
        mag = q.copy()
        for c in range(3):
            if not res.tested[0, c]:
                break
            x = int(inp.draft_tokens[0, c])
            m = int(res.m[0, c])
            A = [x] + [int(t) for t in table[x, 1:m + 1]]
            assert np.isclose(res.qa[0, c], q[A].sum(), rtol=1e-12)
            assert np.isclose(res.qa_mag[0, c], mag[A].sum(), rtol=1e-12), (seed, c)
            assert res.qa_mag[0, c] >= res.qa[0, c] * (1 - 1e-12)
            if c == 0:
                assert np.isclose(res.qa_mag[0, c], res.qa[0, c], rtol=1e-12)
            if res.accept_len[0] > 0 and res.accept_path[0, 0] == c:
                break
            w = q.copy()
            w[x] = q[A].sum()
            w[A[1:]] = 0.0
            w = np.maximum(w - p, 0.0)
            W = w.sum()
            mag = np.where(w > 0, (mag + p) / W, 0.0)
            q = w / W
            p = p.copy()
            p[x] = 0.0
            p = p / p.sum()
            checked += c >= 0
    assert checked > 20          # later siblings were reached
