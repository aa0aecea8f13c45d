"""Seeded synthetic inputs for LANTERN relaxed verification.

This module only *makes inputs*: codebooks, logit rows, draft trees, draft tokens and
uniforms, with the shapes and statistics of the paper's workloads (Section 5.1 and
Appendix B.2: V = 16384 codes, 16x16 / 32x32 token grids, 60 candidate tokens per
verification, classifier-free guidance scales 7.5 / 4.0, tau = 1).  It contains no part
of the verification method itself (no softmax, no neighbourhood, no acceptance rule), so
it can feed both the CPU oracle and the CUDA library without coupling them.

Draft tokens are drawn from the drafter distribution with the Gumbel-max trick (argmax of
logit + Gumbel noise is a softmax sample; the top-c of the perturbed logits is a draw of c
distinct tokens without replacement), which needs no normalised probabilities.

Two back ends produce the same recipe:
  * numpy (Philox counter-based streams) -- used by every test and by the oracle legs;
  * torch on a CUDA device -- used for inputs too large to make on the host in seconds.
The two do not produce the same random stream; any comparison uses one back end's bytes
on both sides.
"""
from __future__ import annotations

import dataclasses
from typing import Optional

import numpy as np

BASE_SEED = 20241003  # date of the paper's first arXiv version; any fixed integer works

F32 = 0
BF16 = 1


# --------------------------------------------------------------------------------------
# bf16 helpers (storage format only: uint16 bit patterns, round-to-nearest-even)
# --------------------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even) and return the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    nan = (u & 0x7FFFFFFF) > 0x7F800000
    r = (u + (0x7FFF + ((u >> 16) & 1))) >> 16
    r = np.where(nan, (u >> 16) | 0x0040, r)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to fp32 exactly."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def _rng(seed: int, stream: int) -> np.random.Generator:
    """One independent Philox stream per (seed, tensor id)."""
    return np.random.Generator(np.random.Philox(key=[np.uint64(seed), np.uint64(stream)]))


# --------------------------------------------------------------------------------------
# codebooks
# --------------------------------------------------------------------------------------
def codebook_gaussian(V: int, D: int, seed: int = BASE_SEED, normalise: bool = True) -> np.ndarray:
    """[V, D] fp32 codebook with N(0,1) entries, rows scaled to unit l2 norm if asked."""
    g = _rng(seed, 1).standard_normal((V, D))
    if normalise:
        g = g / np.sqrt((g * g).sum(axis=1, keepdims=True))
    return g.astype(np.float32)


def codebook_clustered(V: int, D: int, centres: int = 512, sigma: float = 0.1,
                       seed: int = BASE_SEED) -> np.ndarray:
    """[V, D] fp32 codebook: code i = centre[i mod centres] + sigma * N(0, I)."""
    r = _rng(seed, 2)
    c = r.standard_normal((centres, D))
    x = c[np.arange(V) % centres] + sigma * r.standard_normal((V, D))
    return x.astype(np.float32)


def codebook_integer(V: int, D: int, lo: int = -3, hi: int = 4, seed: int = BASE_SEED) -> np.ndarray:
    """[V, D] fp32 codebook with small integer entries: every squared distance is an exact
    integer in any floating-point format, so exact ties occur and orders are unambiguous."""
    return _rng(seed, 3).integers(lo, hi, size=(V, D)).astype(np.float32)


# --------------------------------------------------------------------------------------
# trees
# --------------------------------------------------------------------------------------
def tree_parents(B: int, N: int, depth: int = 6, seed: int = BASE_SEED) -> np.ndarray:
    """[B, N] int32 parent arrays of EAGLE-2-shaped draft trees.

    Nodes 0..depth-1 form a spine of depth 1..depth (node 0 hangs off the root, parent -1).
    Every later node picks its parent uniformly from {root} + {earlier nodes of depth < depth}.
    A parent index is always smaller than the node's own index.
    """
    r = _rng(seed, 4)
    par = np.full((B, N), -1, dtype=np.int32)
    for b in range(B):
        d = np.zeros(N, dtype=np.int64)
        for i in range(N):
            if i < depth:
                par[b, i] = i - 1
            else:
                cand = [-1] + [j for j in range(i) if d[j] < depth]
                par[b, i] = cand[int(r.integers(0, len(cand)))]
            d[i] = 1 if par[b, i] < 0 else d[par[b, i]] + 1
    return par


def chain_parents(B: int, N: int) -> np.ndarray:
    """[B, N] int32 parents of a chain written as a tree: parent(i) = i - 1."""
    return np.tile(np.arange(-1, N - 1, dtype=np.int32), (B, 1))


# --------------------------------------------------------------------------------------
# one verification call
# --------------------------------------------------------------------------------------
@dataclasses.dataclass
class VerifyInputs:
    """Host-side inputs of one verification call, stored exactly as the library reads them."""
    target_logits: np.ndarray          # [C, B, N+1, V]  float32, or uint16 holding bf16 bits
    draft_logits: np.ndarray           # [B, N+1, V]     same storage
    dtype: int                         # F32 | BF16
    cfg_scale: float
    has_uncond: int
    T: float
    draft_tokens: np.ndarray           # [B, N] int32
    tree_parents: Optional[np.ndarray]  # [B, N] int32 or None (chain)
    uniforms: np.ndarray               # [B, N+1] float32 in [0, 1)
    B: int
    N: int
    V: int

    def target_f32(self) -> np.ndarray:
        return self.target_logits if self.dtype == F32 else bf16_bits_to_f32(self.target_logits)

    def draft_f32(self) -> np.ndarray:
        return self.draft_logits if self.dtype == F32 else bf16_bits_to_f32(self.draft_logits)


def _store(x: np.ndarray, dtype: int) -> np.ndarray:
    x = x.astype(np.float32)
    return x if dtype == F32 else f32_to_bf16_bits(x)


def _gumbel(r: np.random.Generator, shape) -> np.ndarray:
    u = r.random(shape)
    u = np.clip(u, 1e-300, 1.0 - 1e-16)
    return -np.log(-np.log(u))


def verify_inputs(B: int, N: int, V: int, *, dtype: int = BF16, has_uncond: bool = True,
                  cfg_scale: float = 7.5, T: float = 1.0, sigma_target: float = 1.0,
                  sigma_draft: float = 0.7, rho: float = 0.0, peaked_frac: float = 0.0,
                  peak_logit: float = 6.0, parents: Optional[np.ndarray] = None,
                  seed: int = BASE_SEED) -> VerifyInputs:
    """Inputs of one call.

    cond ~ N(0, sigma_target^2); uncond = rho*cond + sqrt(1-rho^2)*N(0, sigma_target^2)
    (rho = 0 is the literal independent-rows recipe, rho close to 1 gives the flat
    post-guidance distributions the paper reports for visual AR models).  A fraction
    `peaked_frac` of context rows gets +peak_logit on one token in cond and uncond alike.
    The drafter row is the guided target row (as stored) plus N(0, sigma_draft^2); the
    centre of that noise is the only use of the guidance scale here and merely shapes how
    close drafter and target are.  Children of one context carry distinct tokens drawn
    without replacement from the drafter's row of that context.
    """
    R = N + 1
    r = _rng(seed, 10)
    cond = sigma_target * r.standard_normal((B, R, V))
    if has_uncond:
        unc = rho * cond + np.sqrt(max(0.0, 1.0 - rho * rho)) * sigma_target * r.standard_normal((B, R, V))
    if peaked_frac > 0.0:
        hit = r.random((B, R)) < peaked_frac
        tok = r.integers(0, V, size=(B, R))
        bb, rr = np.nonzero(hit)
        cond[bb, rr, tok[bb, rr]] += peak_logit
        if has_uncond:
            unc[bb, rr, tok[bb, rr]] += peak_logit
    cond_s = _store(cond, dtype)
    if has_uncond:
        unc_s = _store(unc, dtype)
        target = np.stack([cond_s, unc_s], axis=0)
        cw = cond_s if dtype == F32 else bf16_bits_to_f32(cond_s)
        uw = unc_s if dtype == F32 else bf16_bits_to_f32(unc_s)
        centre = uw.astype(np.float64) + float(cfg_scale) * (cw.astype(np.float64) - uw.astype(np.float64))
    else:
        target = cond_s[None]
        centre = (cond_s if dtype == F32 else bf16_bits_to_f32(cond_s)).astype(np.float64)
    draft = _store(centre + sigma_draft * r.standard_normal((B, R, V)), dtype)
    dw = (draft if dtype == F32 else bf16_bits_to_f32(draft)).astype(np.float64) / float(T)

    # tokens: Gumbel-max on the drafter row of the parent context
    par = parents if parents is not None else chain_parents(B, N)
    tokens = np.zeros((B, N), dtype=np.int32)
    g = _rng(seed, 11)
    for b in range(B):
        for c in range(R):  # context c = root (0) or the context after node c-1
            kids = np.nonzero(par[b] == c - 1)[0]
            if kids.size == 0:
                continue
            pert = dw[b, c] + _gumbel(g, V)
            top = np.argpartition(-pert, kids.size - 1)[:kids.size]
            top = top[np.argsort(-pert[top], kind="stable")]
            tokens[b, kids] = top.astype(np.int32)
    uniforms = _rng(seed, 12).random((B, R), dtype=np.float32)
    uniforms = np.minimum(uniforms, np.float32(1.0 - 2.0 ** -24))
    return VerifyInputs(target_logits=np.ascontiguousarray(target), draft_logits=np.ascontiguousarray(draft),
                        dtype=dtype, cfg_scale=float(cfg_scale), has_uncond=int(has_uncond), T=float(T),
                        draft_tokens=tokens, tree_parents=None if parents is None else par.astype(np.int32),
                        uniforms=uniforms, B=B, N=N, V=V)


# --------------------------------------------------------------------------------------
# the five named configurations (shapes and statistics; sizes can be scaled down by tests)
# --------------------------------------------------------------------------------------
CONFIGS = {
    # name: codebook recipe, table parameters, call shape, logit recipe
    "tiny": dict(V=1024, D=8, codebook="gaussian", k=16, delta=0.1, B=1, N=4, tree=False,
                 dtype=F32, has_uncond=False, cfg_scale=1.0, T=1.0, sigma_target=1.5,
                 sigma_draft=0.5, peaked_frac=0.0, steps=64),
    "single_image": dict(V=16384, D=8, codebook="gaussian", k=100, delta=0.2, B=1, N=60, tree=True,
                         dtype=BF16, has_uncond=True, cfg_scale=7.5, T=1.0, sigma_target=1.0,
                         sigma_draft=0.7, peaked_frac=0.0, steps=256),
    "batch_chain": dict(V=16384, D=8, codebook="gaussian", k=1000, delta=0.4, B=32, N=7, tree=False,
                        dtype=BF16, has_uncond=True, cfg_scale=7.5, T=1.0, sigma_target=1.0,
                        sigma_draft=0.7, peaked_frac=0.05, steps=256),
    "px512_tree": dict(V=16384, D=8, codebook="gaussian", k=300, delta=0.3, B=8, N=60, tree=True,
                       dtype=BF16, has_uncond=True, cfg_scale=4.0, T=1.0, sigma_target=1.2,
                       sigma_draft=0.7, peaked_frac=0.0, steps=1024),
    "stress": dict(V=16384, D=256, codebook="clustered", k=1000, delta=0.4, B=128, N=60, tree=True,
                   dtype=BF16, has_uncond=True, cfg_scale=7.5, T=1.0, sigma_target=1.0,
                   sigma_draft=0.7, peaked_frac=0.0, steps=256),
}


def config_codebook(name: str, seed: int = BASE_SEED, V: Optional[int] = None) -> np.ndarray:
    c = CONFIGS[name]
    V = V or c["V"]
    if c["codebook"] == "clustered":
        return codebook_clustered(V, c["D"], seed=seed)
    return codebook_gaussian(V, c["D"], seed=seed, normalise=True)


def config_verify_inputs(name: str, step: int = 0, seed: int = BASE_SEED, B: Optional[int] = None,
                         V: Optional[int] = None, rho: float = 0.0) -> VerifyInputs:
    """Inputs of verification step `step` of a named configuration (B, V can be overridden)."""
    c = CONFIGS[name]
    B = B or c["B"]
    V = V or c["V"]
    s = seed + 1000003 * (step + 1)
    par = tree_parents(B, c["N"], depth=6, seed=s) if c["tree"] else None
    return verify_inputs(B, c["N"], V, dtype=c["dtype"], has_uncond=c["has_uncond"],
                         cfg_scale=c["cfg_scale"], T=c["T"], sigma_target=c["sigma_target"],
                         sigma_draft=c["sigma_draft"], rho=rho, peaked_frac=c["peaked_frac"],
                         parents=par, seed=s)
