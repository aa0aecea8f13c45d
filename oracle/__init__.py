"""ctypes front end of the CPU oracle (oracle/lantern_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests, by the smoke check and by the CPU-baseline /
reference legs of the benchmark.  The CUDA library and its Python binding never import it.
"""
from __future__ import annotations

import ctypes
import dataclasses
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lantern_oracle.cpp")
_LIB = os.path.join(_HERE, "liblantern_oracle.so")

ST_BAD_TOKEN, ST_BAD_PARENT, ST_BAD_UNIFORM, ST_NONFINITE, ST_DEGENERATE, ST_BAD_TABLE = 1, 2, 4, 8, 16, 32
DIV_TVD, DIV_JSD = 0, 1
DEGENERATE_EPS = 1e-5      # reading R10: a residual of total weight <= this defines no distribution


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fused contraction, so fp32 steps round where written)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fPIC", "-shared",
                               "-Wall", "-Wextra", "-o", _LIB, _SRC])
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_count_order_differences.restype = ctypes.c_int64
        _lib.oracle_jsd_collapsed.restype = ctypes.c_double
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def normalize_rows(codebook: np.ndarray) -> np.ndarray:
    """Codes scaled to unit length in the canonical fp32 sequence (cosine variant, Section 5.3.1)."""
    cb = np.ascontiguousarray(codebook, dtype=np.float32)
    out = np.empty_like(cb)
    rc = _load().oracle_normalize_rows(_p(cb), cb.shape[0], cb.shape[1], _p(out))
    if rc != 0:
        raise ValueError(f"oracle_normalize_rows: bad arguments ({rc})")
    return out


def build_neighbors(codebook: np.ndarray, k: int, rows: Optional[np.ndarray] = None, metric: str = "l2"):
    """B_k for every code, or for the codes listed in `rows` (Algorithm 2, precompute block).
    metric "l2" (the paper's choice) or "cosine" (Section 5.3.1: the same routine on unit-length codes).
    Returns idx [n, k] int32, dist [n, k] fp32 with n = V or len(rows)."""
    assert metric in ("l2", "cosine")
    cb = np.ascontiguousarray(codebook, dtype=np.float32)
    if metric == "cosine":
        cb = normalize_rows(cb)
    V, D = cb.shape
    rw = None if rows is None else np.ascontiguousarray(rows, dtype=np.int32)
    n = V if rw is None else rw.shape[0]
    idx = np.empty((n, k), dtype=np.int32)
    dist = np.empty((n, k), dtype=np.float32)
    rc = _load().oracle_build_neighbors_rows(_p(cb), V, D, int(k), _p(rw), n, _p(idx), _p(dist))
    if rc != 0:
        raise ValueError(f"oracle_build_neighbors: bad arguments ({rc})")
    return idx, dist


def count_order_differences(codebook: np.ndarray, idx: np.ndarray) -> int:
    cb = np.ascontiguousarray(codebook, dtype=np.float32)
    V, D = cb.shape
    ix = np.ascontiguousarray(idx, dtype=np.int32)
    return int(_load().oracle_count_order_differences(_p(cb), V, D, ix.shape[1], _p(ix)))


def row_distribution(row_c: np.ndarray, row_u: Optional[np.ndarray], dtype: int, cfg_scale: float,
                     T: float, top_k: int = 0) -> np.ndarray:
    """softmax((l_u + s (l_c - l_u)) / T) of one context row, in double precision; top_k > 0 first
    sets the processed logits below the top_k-th largest to -inf (Appendix B.2)."""
    rc_ = np.ascontiguousarray(row_c)
    ru_ = None if row_u is None else np.ascontiguousarray(row_u)
    V = rc_.shape[0]
    out = np.empty(V, dtype=np.float64)
    rc = _load().oracle_row_distribution_topk(_p(rc_), _p(ru_), int(dtype), int(ru_ is not None),
                                              ctypes.c_float(cfg_scale), ctypes.c_float(T), int(top_k), V, _p(out))
    if rc != 0:
        raise ValueError(f"oracle_row_distribution failed ({rc})")
    return out


def jsd_collapsed(q0: float, S: float) -> float:
    """JSD (natural log) between q and q_{k,delta}(.|D = x~) when A moves mass S onto x~, q(x~) = q0."""
    return float(_load().oracle_jsd_collapsed(ctypes.c_double(q0), ctypes.c_double(S)))


def a_set(q: np.ndarray, nbr_row: np.ndarray, delta: float, divergence: int = DIV_TVD):
    """Size (beyond x~) and moved mass of A_{k,delta}(x~) on distribution q (Algorithm 2, second block);
    the bound is on the TVD (Section 4.3) or on the JSD (Section 5.3.2).  nbr_row[0] is x~."""
    q_ = np.ascontiguousarray(q, dtype=np.float64)
    nb = np.ascontiguousarray(nbr_row, dtype=np.int32)
    moved = ctypes.c_double(0.0)
    margin = ctypes.c_double(0.0)
    bad = ctypes.c_int(0)
    m = _load().oracle_a_set_div(_p(q_), q_.shape[0], _p(nb), nb.shape[0], ctypes.c_double(delta), int(divergence),
                                 ctypes.c_double(q_[nb[0]]), ctypes.byref(moved), ctypes.byref(margin),
                                 ctypes.byref(bad))
    return int(m), moved.value, margin.value


@dataclasses.dataclass
class VerifyResult:
    accept_len: np.ndarray      # [B] int32
    next_token: np.ndarray      # [B] int32
    accept_path: np.ndarray     # [B, N] int32, -1 padded
    status: np.ndarray          # [B] int32 bit flags
    tested: np.ndarray          # [B, N] uint8
    qa: np.ndarray              # [B, N] float64: sum of the current target over A_{k,delta}(x~)
    px: np.ndarray              # [B, N] float64: current drafter probability of x~
    m: np.ndarray               # [B, N] int32: |A_{k,delta}(x~)| - 1, -1 if untested
    margin: np.ndarray          # [B, N] float64: distance of the node's decisions to flipping
    w: np.ndarray               # [B] float64: total weight of the last residual
    draw_margin: np.ndarray     # [B] float64
    qa_mag: np.ndarray          # [B, N] float64: magnitude of the terms qa was formed from (>= qa)


def verify(target_logits: np.ndarray, draft_logits: np.ndarray, dtype: int, cfg_scale: float, has_uncond: int,
           T: float, draft_tokens: np.ndarray, tree_parents: Optional[np.ndarray], neighbor_idx: np.ndarray,
           delta: float, uniforms: np.ndarray, divergence: int = DIV_TVD, top_k: int = 0,
           degenerate_eps: float = DEGENERATE_EPS) -> VerifyResult:
    """One verification call on host arrays (same layouts as the library's lantern_verify).
    degenerate_eps: total weight at or below which a residual counts as undefined (reading R10)."""
    tl = np.ascontiguousarray(target_logits)
    dl = np.ascontiguousarray(draft_logits)
    C, B, R, V = tl.shape
    N = R - 1
    assert C == (2 if has_uncond else 1)
    assert dl.shape == (B, R, V)
    want = np.float32 if dtype == 0 else np.uint16
    assert tl.dtype == want and dl.dtype == want
    tok = np.ascontiguousarray(draft_tokens, dtype=np.int32).reshape(B, N)
    par = None if tree_parents is None else np.ascontiguousarray(tree_parents, dtype=np.int32).reshape(B, N)
    nb = np.ascontiguousarray(neighbor_idx, dtype=np.int32)
    assert nb.shape[0] == V
    k = nb.shape[1]
    un = np.ascontiguousarray(uniforms, dtype=np.float32).reshape(B, R)
    res = VerifyResult(
        accept_len=np.zeros(B, np.int32), next_token=np.zeros(B, np.int32),
        accept_path=np.full((B, N), -1, np.int32), status=np.zeros(B, np.int32),
        tested=np.zeros((B, N), np.uint8), qa=np.zeros((B, N)), px=np.zeros((B, N)),
        m=np.full((B, N), -1, np.int32), margin=np.full((B, N), np.inf), w=np.zeros(B),
        draw_margin=np.full(B, np.inf), qa_mag=np.zeros((B, N)))
    rc = _load().oracle_verify_ex(
        _p(tl), _p(dl), int(dtype), ctypes.c_float(cfg_scale), int(has_uncond), ctypes.c_float(T), _p(tok),
        _p(par), _p(nb), int(k), ctypes.c_float(delta), int(divergence), int(top_k), _p(un), B, N, V,
        _p(res.accept_len),
        _p(res.next_token), _p(res.accept_path), _p(res.status), _p(res.tested), _p(res.qa), _p(res.px),
        _p(res.m), _p(res.margin), _p(res.w), _p(res.draw_margin), _p(res.qa_mag), ctypes.c_double(degenerate_eps))
    if rc != 0:
        raise ValueError(f"oracle_verify: bad arguments ({rc})")
    return res


def verify_inputs(inp, neighbor_idx: np.ndarray, delta: float, divergence: int = DIV_TVD,
                  top_k: int = 0, degenerate_eps: float = DEGENERATE_EPS) -> VerifyResult:
    """Convenience: run `verify` on a lantern_inputs.VerifyInputs bundle."""
    return verify(inp.target_logits, inp.draft_logits, inp.dtype, inp.cfg_scale, inp.has_uncond, inp.T,
                  inp.draft_tokens, inp.tree_parents, neighbor_idx, delta, inp.uniforms, divergence, top_k,
                  degenerate_eps)


@dataclasses.dataclass
class GreedyResult:
    accept_len: np.ndarray      # [B] int32
    next_token: np.ndarray      # [B] int32
    accept_path: np.ndarray     # [B, N] int32, -1 padded
    status: np.ndarray          # [B] int32 bit flags
    tested: np.ndarray          # [B, N] uint8
    qa: np.ndarray              # [B, N] float64: sum of the target over A_{k,delta}(x~)
    m: np.ndarray               # [B, N] int32
    margin: np.ndarray          # [B, N] float64: distance of the node's decisions to flipping


def verify_greedy(target_logits: np.ndarray, dtype: int, cfg_scale: float, has_uncond: int,
                  draft_tokens: np.ndarray, tree_parents: Optional[np.ndarray], neighbor_idx: np.ndarray,
                  delta: float, divergence: int = DIV_TVD, top_k: int = 0) -> GreedyResult:
    """Greedy-decoding verification (Section 4.3, last sentence) on host arrays."""
    tl = np.ascontiguousarray(target_logits)
    C, B, R, V = tl.shape
    N = R - 1
    assert C == (2 if has_uncond else 1)
    assert tl.dtype == (np.float32 if dtype == 0 else np.uint16)
    tok = np.ascontiguousarray(draft_tokens, dtype=np.int32).reshape(B, N)
    par = None if tree_parents is None else np.ascontiguousarray(tree_parents, dtype=np.int32).reshape(B, N)
    nb = np.ascontiguousarray(neighbor_idx, dtype=np.int32)
    assert nb.shape[0] == V
    res = GreedyResult(accept_len=np.zeros(B, np.int32), next_token=np.zeros(B, np.int32),
                       accept_path=np.full((B, N), -1, np.int32), status=np.zeros(B, np.int32),
                       tested=np.zeros((B, N), np.uint8), qa=np.zeros((B, N)), m=np.full((B, N), -1, np.int32),
                       margin=np.full((B, N), np.inf))
    rc = _load().oracle_verify_greedy_ex(_p(tl), int(dtype), ctypes.c_float(cfg_scale), int(has_uncond), _p(tok),
                                         _p(par), _p(nb), int(nb.shape[1]), ctypes.c_float(delta), int(divergence),
                                         int(top_k), B, N, V, _p(res.accept_len),
                                      _p(res.next_token), _p(res.accept_path), _p(res.status), _p(res.tested),
                                      _p(res.qa), _p(res.m), _p(res.margin))
    if rc != 0:
        raise ValueError(f"oracle_verify_greedy: bad arguments ({rc})")
    return res


def aggregate_all(rows_c: np.ndarray, rows_u: Optional[np.ndarray], dtype: int, cfg_scale: float, T: float,
                  neighbor_idx: np.ndarray, delta: float):
    """agg[r, x] = sum of row r's distribution over A_{k,delta}(x), for every token x (a benchmark of the
    V x k gather-sum; the paper's method needs it for the drafted tokens only).  Returns (agg, m, margin)."""
    rc_ = np.ascontiguousarray(rows_c)
    ru_ = None if rows_u is None else np.ascontiguousarray(rows_u)
    rows, V = rc_.shape
    nb = np.ascontiguousarray(neighbor_idx, dtype=np.int32)
    agg = np.empty((rows, V), np.float64)
    m = np.empty((rows, V), np.int32)
    margin = np.empty((rows, V), np.float64)
    rc = _load().oracle_aggregate_all(_p(rc_), _p(ru_), int(dtype), int(ru_ is not None), ctypes.c_float(cfg_scale),
                                      ctypes.c_float(T), _p(nb), int(nb.shape[1]), ctypes.c_float(delta), rows, V,
                                      _p(agg), _p(m), _p(margin))
    if rc != 0:
        raise ValueError(f"oracle_aggregate_all failed ({rc})")
    return agg, m, margin
