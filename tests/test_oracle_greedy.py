"""Pins of the oracle's greedy-decoding verification (Section 4.3, last sentence).

  * k = 1 or delta = 0: plain greedy speculative decoding -- a draft is accepted iff it is the
    target's arg max, and the emitted token is always the target's arg max;
  * definition by brute force: build q_{k,delta}(.|D = x~) as Section 4.3 writes it and take numpy's
    arg max (x~ wins ties);
  * the relaxed rule accepts whenever the plain rule does, and more as delta or k grow;
  * large delta: the whole neighbourhood B_k is aggregated (eq. 1's numerator);
  * chain written as a tree gives the same result; the walk follows parents.
"""
import numpy as np
import pytest

import lantern_inputs as li
import oracle


def np_softmax(z):
    z = np.asarray(z, dtype=np.float64)
    e = np.exp(z - z.max())
    return e / e.sum()


def case(B, N, V, seed, parents=None, **kw):
    return li.verify_inputs(B, N, V, dtype=li.BF16, has_uncond=True, cfg_scale=kw.pop("cfg_scale", 2.0),
                            sigma_target=1.0, sigma_draft=kw.pop("sigma_draft", 0.3), rho=0.9, parents=parents,
                            seed=seed, **kw)


def run(inp, table, delta):
    return oracle.verify_greedy(inp.target_logits, inp.dtype, inp.cfg_scale, inp.has_uncond, inp.draft_tokens,
                                inp.tree_parents, table, delta)


def q_row(inp, b, t):
    return oracle.row_distribution(inp.target_logits[0, b, t], inp.target_logits[1, b, t], inp.dtype, inp.cfg_scale, 1.0)


@pytest.mark.parametrize("mode", ["k1", "delta0"])
def test_reduces_to_plain_greedy(mode):
    V, N, B = 128, 6, 150
    inp = case(B, N, V, seed=7)
    if mode == "k1":
        table, delta = np.arange(V, dtype=np.int32)[:, None], 0.3
    else:
        table, delta = oracle.build_neighbors(li.codebook_gaussian(V, 4, seed=2), 9)[0], 0.0
    res = run(inp, table, delta)
    n_full = 0
    for b in range(B):
        al = 0
        for t in range(N):
            q = q_row(inp, b, t)
            if q[inp.draft_tokens[b, t]] < q.max():     # not an arg max (bf16 logits do tie: ties accept)
                break
            al += 1
        assert res.accept_len[b] == al
        assert res.next_token[b] == int(np.argmax(q_row(inp, b, al)))
        n_full += al == N
    assert 0 < (res.accept_len > 0).sum() < B and np.all(res.status == 0)


@pytest.mark.parametrize("delta", [0.02, 0.1, 0.4])
def test_definition_by_brute_force(delta):
    V, k = 256, 24
    table = oracle.build_neighbors(li.codebook_gaussian(V, 8, seed=4), k)[0]
    inp = case(60, 5, V, seed=11, sigma_draft=0.8)
    res = run(inp, table, delta)
    seen = acc = 0
    for b in range(inp.B):
        for t in range(inp.N):
            if not res.tested[b, t]:
                continue
            seen += 1
            q = q_row(inp, b, t)
            x = inp.draft_tokens[b, t]
            A = table[x, : res.m[b, t] + 1]
            qd = q.copy()
            qd[A] = 0.0
            qd[x] = q[A].sum()                      # q_{k,delta}(.|D = x~) of Section 4.3
            assert 0.5 * np.abs(qd - q).sum() < float(np.float32(delta))
            want = bool(qd[x] >= qd.max())          # x~ is an arg max (ties go to x~)
            got = bool(res.accept_len[b] > t)
            assert got == want
            acc += got
            if not got:
                assert res.next_token[b] == int(np.argmax(qd)) == int(np.argmax(q))
    assert seen > inp.B and 0 < acc < seen


def test_monotone_in_delta_and_k():
    V, k = 256, 32
    table = oracle.build_neighbors(li.codebook_gaussian(V, 8, seed=4), k)[0]
    inp = case(80, 1, V, seed=13, sigma_draft=1.0)
    prev = None
    for delta in (0.0, 0.05, 0.2, 0.5, 2.0):
        a = run(inp, table, delta).accept_len
        if prev is not None:
            assert np.all(a >= prev)
        prev = a
    prev = None
    for kk in (1, 4, 16, 32):
        a = run(inp, np.ascontiguousarray(table[:, :kk]), 0.3).accept_len
        if prev is not None:
            assert np.all(a >= prev)
        prev = a
    full = run(inp, table, 2.0)
    for b in range(inp.B):
        q = q_row(inp, b, 0)
        x = inp.draft_tokens[b, 0]
        assert full.m[b, 0] == k - 1 and abs(full.qa[b, 0] - q[table[x]].sum()) < 1e-12


def test_trees():
    V, k = 256, 16
    table = oracle.build_neighbors(li.codebook_gaussian(V, 8, seed=4), k)[0]
    par = li.tree_parents(40, 20, depth=4, seed=9)
    inp = case(40, 20, V, seed=17, parents=par, sigma_draft=0.5)
    res = run(inp, table, 0.3)
    assert res.accept_len.max() >= 2
    for b in range(40):
        prev = -1
        for d in range(res.accept_len[b]):
            node = res.accept_path[b, d]
            assert par[b, node] == prev and res.tested[b, node]
            prev = node
        q = q_row(inp, b, prev + 1)
        assert res.next_token[b] == int(np.argmax(q))
    chain = case(30, 6, V, seed=19)
    a = run(chain, table, 0.3)
    import dataclasses
    b_ = run(dataclasses.replace(chain, tree_parents=li.chain_parents(30, 6)), table, 0.3)
    for f in ("accept_len", "next_token", "accept_path", "tested", "qa", "m"):
        assert np.array_equal(getattr(a, f), getattr(b_, f)), f
