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
that magnitude as qa_mag).
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
    for u, d in trials:
        r = oracle.verify_inputs(dataclasses.replace(one, uniforms=u), table, max(d, 0.0), divergence, top_k)
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
    near = outside = degenerate = 0
    bad = []
    st_mask = np.ones(inp.B, bool)
    for b in range(inp.B):
        same = (g_len[b] == ora.accept_len[b] and g_tok[b] == ora.next_token[b]
                and np.array_equal(g_path[b], ora.accept_path[b]))
        if same:
            continue
        # A residual whose total weight is exactly zero in double precision (possible only when the
        # drafted token lies outside the drafter's own support, e.g. cut by the top-k filter, and target
        # and drafter agree elsewhere) is rounding noise in fp32: the library may report it or draw
        # from the noise; the walk up to that point must still agree.
        if (ora.status[b] & oracle.ST_DEGENERATE) and g_len[b] == ora.accept_len[b] \
                and np.array_equal(g_path[b], ora.accept_path[b]) and (g_st[b] & ~oracle.ST_DEGENERATE) == 0:
            degenerate += 1
            st_mask[b] = False
            continue
        if _explained_by_window(inp, table, delta, b, ora, (g_len[b], g_tok[b], g_path[b]), divergence, top_k):
            near += 1
        else:
            outside += 1
            bad.append(b)
    res = dict(n_seq=inp.B, near=near, mismatch_outside=outside, bad=bad, degenerate=degenerate,
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
        rel_px = np.abs(px[t] - ora.px[t]) / np.maximum(ora.px[t], 1e-30)
        res["qa_rel_max"] = float(rel_qa.max()) if rel_qa.size else 0.0
        res["px_rel_max"] = float(rel_px.max()) if rel_px.size else 0.0
        res["nodes_tested"] = int(t.sum())
    return res


def assert_parity(res):
    assert res["mismatch_outside"] == 0, res
    assert res["status_equal"], res
    if "qa_rel_max" in res:
        assert res["m_mismatch_outside"] == 0, res
        assert res["qa_rel_max"] < REL and res["px_rel_max"] < REL, res
