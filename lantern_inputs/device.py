"""The same input recipes as lantern_inputs.verify_inputs, generated with torch on a CUDA device.

For calls too large to make on the host in seconds (thousands of sequences x 16384-wide rows).
The random stream differs from the numpy back end; any comparison with the CPU oracle copies
the device bytes back to the host, so both sides still see identical inputs.  Like the numpy
module this file only makes inputs: tokens are Gumbel-max draws, no probabilities are formed.
"""
from __future__ import annotations

from typing import Optional

import numpy as np
import torch

from . import BASE_SEED, BF16, F32, CONFIGS, VerifyInputs, tree_parents


def verify_inputs_device(B: int, N: int, V: int, *, dtype: int = BF16, has_uncond: bool = True,
                         cfg_scale: float = 7.5, T: float = 1.0, sigma_target: float = 1.0,
                         sigma_draft: float = 0.7, rho: float = 0.0, peaked_frac: float = 0.0,
                         peak_logit: float = 6.0, parents: Optional[np.ndarray] = None,
                         seed: int = BASE_SEED, device: str = "cuda", chunk: int = 128) -> dict:
    """Returns a dict of device tensors with the argument names of the library's verify()."""
    R = N + 1
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(int(seed))
    tdt = torch.bfloat16 if dtype == BF16 else torch.float32
    C = 2 if has_uncond else 1
    target = torch.empty((C, B, R, V), dtype=tdt, device=dev)
    draft = torch.empty((B, R, V), dtype=tdt, device=dev)
    tokens = torch.zeros((B, N), dtype=torch.int32, device=dev)

    if parents is None:
        par = np.tile(np.arange(-1, N - 1, dtype=np.int32), (B, 1))
    else:
        par = np.asarray(parents, dtype=np.int32)
    # rank of each node among the children of its parent (children are tried in node order)
    rank = np.zeros((B, N), dtype=np.int64)
    max_kids = 1
    for b in range(B if parents is not None else 1):
        seen = {}
        for i in range(N):
            p_ = int(par[b, i])
            rank[b, i] = seen.get(p_, 0)
            seen[p_] = rank[b, i] + 1
        if seen:
            max_kids = max(max_kids, max(seen.values()))
    if parents is None:
        rank[:] = 0
    ctx_of = torch.from_numpy(par.astype(np.int64) + 1).to(dev)       # context row a node is tested in
    rank_t = torch.from_numpy(rank).to(dev)

    for b0 in range(0, B, chunk):
        b1 = min(B, b0 + chunk)
        n = b1 - b0
        cond = sigma_target * torch.randn((n, R, V), generator=g, device=dev)
        if has_uncond:
            unc = rho * cond + (max(0.0, 1.0 - rho * rho) ** 0.5) * sigma_target * \
                torch.randn((n, R, V), generator=g, device=dev)
        if peaked_frac > 0.0:
            hit = torch.rand((n, R), generator=g, device=dev) < peaked_frac
            tok = torch.randint(0, V, (n, R), generator=g, device=dev)
            bump = torch.zeros((n, R, V), device=dev)
            bump.scatter_(2, tok[..., None], hit[..., None].float() * peak_logit)
            cond += bump
            if has_uncond:
                unc += bump
            del bump
        target[0, b0:b1] = cond.to(tdt)
        if has_uncond:
            target[1, b0:b1] = unc.to(tdt)
            cw, uw = target[0, b0:b1].float(), target[1, b0:b1].float()
            centre = uw + cfg_scale * (cw - uw)       # only centres the drafter's noise (workload shaping)
        else:
            centre = target[0, b0:b1].float()
        draft[b0:b1] = (centre + sigma_draft * torch.randn((n, R, V), generator=g, device=dev)).to(tdt)
        if N > 0:
            u = torch.rand((n, R, V), generator=g, device=dev).clamp_(1e-20, 1.0 - 1e-7)
            pert = draft[b0:b1].float() / T - torch.log(-torch.log(u))
            top = torch.topk(pert, max_kids, dim=2).indices          # [n, R, max_kids], distinct per context
            flat = top.reshape(n, R * max_kids)
            sel = ctx_of[b0:b1] * max_kids + rank_t[b0:b1]
            tokens[b0:b1] = torch.gather(flat, 1, sel).to(torch.int32)
            del u, pert, top
        del cond, centre
    uniforms = torch.rand((B, R), generator=g, device=dev, dtype=torch.float32).clamp_(0.0, 1.0 - 2.0 ** -24)
    return dict(target_logits=target, draft_logits=draft, dtype=dtype, cfg_scale=float(cfg_scale),
                has_uncond=int(has_uncond), T=float(T), draft_tokens=tokens,
                tree_parents=None if parents is None else torch.from_numpy(par).to(dev),
                uniforms=uniforms, B=B, N=N, V=V)


def config_verify_inputs_device(name: str, B: Optional[int] = None, seed: int = BASE_SEED, rho: float = 0.0,
                                device: str = "cuda") -> dict:
    c = CONFIGS[name]
    B = B or c["B"]
    par = tree_parents(B, c["N"], depth=6, seed=seed) if c["tree"] else None
    return verify_inputs_device(B, c["N"], c["V"], dtype=c["dtype"], has_uncond=c["has_uncond"],
                                cfg_scale=c["cfg_scale"], T=c["T"], sigma_target=c["sigma_target"],
                                sigma_draft=c["sigma_draft"], rho=rho, peaked_frac=c["peaked_frac"],
                                parents=par, seed=seed, device=device)


def to_host(d: dict, rows: Optional[np.ndarray] = None) -> VerifyInputs:
    """Copy (a subset of the sequences of) a device bundle back into a host VerifyInputs."""
    sel = slice(None) if rows is None else torch.as_tensor(rows, device=d["target_logits"].device)

    def bits(t):
        t = t.contiguous()
        if t.dtype == torch.bfloat16:
            return t.view(torch.int16).cpu().numpy().view(np.uint16)
        return t.cpu().numpy()
    tl = bits(d["target_logits"][:, sel])
    dl = bits(d["draft_logits"][sel])
    B = dl.shape[0]
    return VerifyInputs(target_logits=tl, draft_logits=dl, dtype=d["dtype"], cfg_scale=d["cfg_scale"],
                        has_uncond=d["has_uncond"], T=d["T"], draft_tokens=d["draft_tokens"][sel].cpu().numpy(),
                        tree_parents=None if d["tree_parents"] is None else d["tree_parents"][sel].cpu().numpy(),
                        uniforms=d["uniforms"][sel].cpu().numpy(), B=B, N=d["N"], V=d["V"])
