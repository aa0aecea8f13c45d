"""Comparison of the CUDA library with the CPU oracle on one verification call.

Rule: accept lengths, next tokens and accepted paths must be identical, except for sequences
in which some decision of the oracle lies within WINDOW of its threshold (the accept test
|r - sum_A q / p(x~)|, the prefix cut |moved mass - delta|, or the final draw's distance to a
CDF edge).  Such a sequence is counted as "near" and must reproduce exactly under the oracle
once the corresponding input (that node's uniform, delta, or the final uniform) is nudged
across the window.  Probabilities must agree to REL: p(x~) relative to itself; sum_A q relative
to the magnitude of the terms it was formed from -- for the first child of a context that is
sum_A q itself, after sibling rejections the target is a difference (q' - p') / W evaluated in
fp32, whose rounding error scales with q' + p', not with the difference (the oracle reports
that magnitude as qa_mag; tests/test_oracle_verify.py pins it against a numpy replay).  The plain
error relative to sum_A q itself is reported beside it (qa_rel_plain_max).

The neighbour table the oracle reads is the ORACLE's: `oracle_table` builds, with the oracle, the
rows that a call's drafted tokens name, and checks them against the library's table.
"""
from __future__ import annotations

import dataclasses

import numpy as np
import torch

import lantern_inputs as li
import oracle
import paper_2410_03355_b200 as lt

WINDOW = 1e-6
REL = 1e-5

_row_cache = {}


def _content_key(codebook: np.ndarray):
    import zlib
    return (codebook.shape, zlib.crc32(np.ascontiguousarray(codebook).tobytes()))


def oracle_table(codebook: np.ndarray, k: int, tokens, device_table=None, metric="l2") -> np.ndarray:
    """[V, k] host table whose rows for `tokens` (any integer array) are built by the oracle; the other
    rows hold -1 beyond the token itself, so that a read the walk should not make shows up as a table fault.
    With `device_table`, asserts that the library's rows for those tokens are identical."""
    V = codebook.shape[0]
    key = (_content_key(codebook), k, metric)
    cache = _row_cache.setdefault(key, {})
    need = np.unique(np.asarray(tokens).ravel())
    need = need[(need >= 0) & (need < V)]
    miss = np.array([t for t in need if int(t) not in cache], dtype=np.int32)
    if miss.size:
        idx, _ = oracle.build_neighbors(codebook, k, rows=miss, metric=metric)
        for r, t in enumerate(miss):
            cache[int(t)] = idx[r]
    tab = np.full((V, k), -1, np.int32)
    tab[:, 0] = np.arange(V)
    for t in need:
        tab[t] = cache[int(t)]
    if device_table is not None and need.size:
        got = device_table[torch.from_numpy(need.astype(np.int64)).to(device_table.device)].cpu().numpy()
        assert np.array_equal(got, tab[need]), "library and oracle neighbour rows differ"
    return tab


def to_device(inp: li.VerifyInputs, device="cuda"):
    def logits(a):
        t = torch.from_numpy(a)
        if inp.dtype == li.BF16:
            t = t.view(torch.int16).view(torch.bfloat16)
        return t.to(device)
    return dict(
        target_logits=logits(inp.target_logits), draft_logits=logits(inp.draft_logits),
        draft_tokens=torch.from_numpy(inp.draft_tokens).to(device),
        tree_parents=None if inp.tree_parents is None else torch.from_numpy(inp.tree_parents).to(device),
        uniforms=torch.from_numpy(inp.uniforms).to(device))


_dev_tables = {}


def tables(codebook: np.ndarray, k: int, tokens):
    """(host table for the oracle, device table for the library) of a codebook.  Up to 2048 codes both are
    the oracle's full table.  Beyond that the device table is the library's own build, and the host table
    holds the oracle's rows for `tokens` (a call's drafted tokens), checked against the library's rows."""
    V = codebook.shape[0]
    key = (_content_key(codebook), k)
    if key not in _dev_tables:
        if V <= 2048:
            host = oracle.build_neighbors(codebook, k)[0]
            _dev_tables[key] = (codebook, host, torch.from_numpy(host).cuda())
        else:
            dev = lt.build_neighbors(torch.from_numpy(codebook).cuda(), k, with_dist=False)[0]
            torch.cuda.synchronize()
            _dev_tables[key] = (codebook, None, dev)
    _, host, dev = _dev_tables[key]
    if host is None:
        host = oracle_table(codebook, k, tokens, dev)
    return host, dev


DIV_NAME = {oracle.DIV_TVD: "tvd", oracle.DIV_JSD: "jsd"}


def run_gpu(inp: li.VerifyInputs, table_dev: torch.Tensor, delta: float, trace=True, divergence=oracle.DIV_TVD,
            top_k=0) -> lt.VerifyOutputs:
    d = to_device(inp)
    out = lt.verify(d["target_logits"], d["draft_logits"], inp.cfg_scale, inp.T, d["draft_tokens"],
                    d["tree_parents"], table_dev, delta, d["uniforms"], trace=trace,
                    divergence=DIV_NAME[divergence], top_k=top_k)
    torch.cuda.synchronize()
    return out


def _slice(inp: li.VerifyInputs, b: int) -> li.VerifyInputs:
    return dataclasses.replace(
        inp, target_logits=np.ascontiguousarray(inp.target_logits[:, b:b + 1]),
        draft_logits=np.ascontiguousarray(inp.draft_logits[b:b + 1]),
        draft_tokens=np.ascontiguousarray(inp.draft_tokens[b:b + 1]),
        tree_parents=None if inp.tree_parents is None else np.ascontiguousarray(inp.tree_parents[b:b + 1]),
        uniforms=inp.uniforms[b:b + 1].copy(), B=1)


def _explained_by_window(inp, table, delta, b, ora, want, divergence=oracle.DIV_TVD, top_k=0) -> bool:
    """Does the oracle give `want` = (len, token, path) once a near-threshold input is nudged?"""
    one = _slice(inp, b)
    eps = 4 * WINDOW
    trials = []
    near_nodes = [i for i in range(inp.N) if ora.tested[b, i] and ora.margin[b, i] < WINDOW]
    for i in near_nodes:
        for s in (-eps, eps):
            u = one.uniforms.copy()
            u[0, i] = np.float32(min(max(u[0, i] + s, 0.0), 1.0 - 2.0 ** -24))
            trials.append((u, delta))
    if near_nodes:
        trials += [(one.uniforms, delta - eps), (one.uniforms, delta + eps)]
    if ora.draw_margin[b] < WINDOW:
        for s in (-eps, eps):
            u = one.uniforms.copy()
            u[0, inp.N] = np.float32(min(max(u[0, inp.N] + s, 0.0), 1.0 - 2.0 ** -24))
            trials.append((u, delta))
    trials = [(u, d, oracle.DEGENERATE_EPS) for u, d in trials]
    if near_nodes:      # a residual's weight within the window of the threshold that makes it degenerate
        trials += [(one.uniforms, delta, oracle.DEGENERATE_EPS - eps), (one.uniforms, delta, oracle.DEGENERATE_EPS + eps)]
    for u, d, e in trials:
        r = oracle.verify_inputs(dataclasses.replace(one, uniforms=u), table, max(d, 0.0), divergence, top_k, e)
        if (r.accept_len[0], r.next_token[0]) == want[:2] and np.array_equal(r.accept_path[0], want[2]):
            return True
    return False


def compare(inp: li.VerifyInputs, table: np.ndarray, delta: float, gpu: lt.VerifyOutputs, ora=None,
            divergence=oracle.DIV_TVD, top_k=0):
    """Returns dict(n_seq, near, mismatch_outside, prob_bad, ...); asserts nothing itself.  With the JSD
    bound the cut's margin is in JSD units (the oracle reports it so); the nudge of delta is the same."""
    if ora is None:
        ora = oracle.verify_inputs(inp, table, delta, divergence, top_k)
    g_len = gpu.accept_len.cpu().numpy()
    g_tok = gpu.next_token.cpu().numpy()
    g_path = gpu.accept_path.cpu().numpy()
    g_st = gpu.status.cpu().numpy()
    near = outside = 0
    bad = []
    st_mask = np.ones(inp.B, bool)
    for b in range(inp.B):
        same = (g_len[b] == ora.accept_len[b] and g_tok[b] == ora.next_token[b]
                and np.array_equal(g_path[b], ora.accept_path[b]))
        if same:
            continue
        st_mask[b] = False     # a different path may meet different faults; the path itself is judged here
        if _explained_by_window(inp, table, delta, b, ora, (g_len[b], g_tok[b], g_path[b]), divergence, top_k):
            near += 1
        else:
            outside += 1
            bad.append(b)
    res = dict(n_seq=inp.B, near=near, mismatch_outside=outside, bad=bad,
               degenerate=int(((ora.status & oracle.ST_DEGENERATE) != 0).sum()),
               status_equal=bool(np.array_equal(g_st[st_mask], ora.status[st_mask])),
               accept_mean=float(ora.accept_len.mean()))
    if gpu.node_qa is not None:
        qa, px, m = gpu.node_qa.cpu().numpy(), gpu.node_px.cpu().numpy(), gpu.node_m.cpu().numpy()
        t = ora.tested.astype(bool) & (ora.status[:, None] == 0)
        far = t & (ora.margin >= WINDOW)
        # A different cut changes sum_A q legitimately, so probabilities are compared where the cut agrees
        # (which it must, away from the window).
        res["m_mismatch_outside"] = int((m[far] != ora.m[far]).sum())
        agree = t & (m == ora.m)
        rel_qa = np.abs(qa[agree] - ora.qa[agree]) / np.maximum(ora.qa_mag[agree], 1e-30)
        rel_plain = np.abs(qa[agree] - ora.qa[agree]) / np.maximum(ora.qa[agree], 1e-30)
        rel_px = np.abs(px[t] - ora.px[t]) / np.maximum(ora.px[t], 1e-30)
        res["qa_rel_max"] = float(rel_qa.max()) if rel_qa.size else 0.0
        res["qa_rel_plain_max"] = float(rel_plain.max()) if rel_plain.size else 0.0
        # first children of their context: no residual round behind them, so the plain relative error binds
        first = agree & (np.abs(ora.qa_mag - ora.qa) <= 1e-12 * np.maximum(ora.qa, 1e-300))
        rel_first = np.abs(qa[first] - ora.qa[first]) / np.maximum(ora.qa[first], 1e-30)
        res["qa_rel_first_max"] = float(rel_first.max()) if rel_first.size else 0.0
        res["px_rel_max"] = float(rel_px.max()) if rel_px.size else 0.0
        res["nodes_tested"] = int(t.sum())
    return res


def assert_parity(res):
    assert res["mismatch_outside"] == 0, res
    assert res["status_equal"], res
    if "qa_rel_max" in res:
        assert res["m_mismatch_outside"] == 0, res
        assert res["qa_rel_max"] < REL and res["px_rel_max"] < REL and res["qa_rel_first_max"] < REL, res


def near_ceiling(n_seq: int) -> int:
    """Most sequences of a call that may sit within the window of a threshold: the windows are 1e-6 wide and a
    sequence takes a few dozen decisions, so more than a handful in a call means a tolerance problem."""
    return max(2, n_seq // 50)
