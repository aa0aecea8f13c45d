"""ctypes binding of liblantern.so: argument marshalling only.

Functions mirror the C entry points of include/lantern.h.  Tensors must live on a CUDA device;
there is no CPU path: a missing library or a CPU tensor raises.
"""
from __future__ import annotations

import ctypes
import dataclasses
import os
from typing import Optional

import torch

F32, BF16 = 0, 1
ST_BAD_TOKEN, ST_BAD_PARENT, ST_BAD_UNIFORM, ST_NONFINITE, ST_DEGENERATE, ST_BAD_TABLE, ST_INTERNAL = \
    1, 2, 4, 8, 16, 32, 64

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "liblantern.so")
_lib = None


class LanternError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (code {code})")


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Load liblantern.so (built in-tree by paper_2410_03355_b200.build). Fails loudly if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise FileNotFoundError(
            f"{_LIB_PATH} not found: build it with `python -m paper_2410_03355_b200.build` "
            "(there is no fallback implementation)")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i32, f32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    lib.lantern_status_string.restype = ctypes.c_char_p
    lib.lantern_status_string.argtypes = [i32]
    lib.lantern_build_workspace_bytes.restype = sz
    lib.lantern_build_workspace_bytes.argtypes = [i32, i32, i32]
    lib.lantern_build_neighbors.restype = i32
    lib.lantern_build_neighbors.argtypes = [vp, i32, i32, i32, vp, vp, vp, sz, vp]
    lib.lantern_verify_workspace_bytes.restype = sz
    lib.lantern_verify_workspace_bytes.argtypes = [i32, i32, i32, i32, i32]
    lib.lantern_last_status.restype = i32
    lib.lantern_last_status.argtypes = [vp, vp, vp]
    lib.lantern_verify_counts.restype = i32
    lib.lantern_verify_counts.argtypes = [vp, vp, vp]
    lib.lantern_debug_wait_test.restype = i32
    lib.lantern_debug_wait_test.argtypes = [i32, i32]
    lib.lantern_build_workspace_bytes_metric.restype = sz
    lib.lantern_build_workspace_bytes_metric.argtypes = [i32, i32, i32, i32]
    lib.lantern_build_neighbors_metric.restype = i32
    lib.lantern_build_neighbors_metric.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, sz, vp]
    lib.lantern_verify_workspace_bytes_ex.restype = sz
    lib.lantern_verify_workspace_bytes_ex.argtypes = [i32, i32, i32, i32, i32, i32]
    lib.lantern_aggregate_all.restype = i32
    lib.lantern_aggregate_all.argtypes = [vp, i32, f32, i32, f32, vp, i32, f32, i32, i32, vp, vp, vp, vp]
    lib.lantern_verify_ex.restype = i32
    lib.lantern_verify_ex.argtypes = [vp, vp, i32, f32, i32, f32, vp, vp, vp, i32, f32, i32, i32, vp, i32, i32, i32,
                                      vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.lantern_kernel_revision.restype = i32
    lib.lantern_kernel_revision.argtypes = []
    lib.lantern_verify_launch_count.restype = i32
    lib.lantern_verify_launch_count.argtypes = [i32, i32]
    lib.lantern_verify_static.restype = i32
    lib.lantern_verify_static.argtypes = [vp, vp, i32, f32, i32, f32, vp, vp, vp, i32, f32, vp, i32, i32, i32,
                                          vp, vp, vp, vp, vp, vp, vp, vp]
    lib.lantern_verify_profile_events.restype = i32
    lib.lantern_verify_profile_events.argtypes = [vp, vp]
    lib.lantern_verify.restype = i32
    lib.lantern_verify.argtypes = [vp, vp, i32, f32, i32, f32, vp, vp, vp, i32, f32, vp, i32, i32, i32,
                                   vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().lantern_status_string(int(code)).decode()


def _ptr(t: Optional[torch.Tensor], dtype=None, name: str = "tensor"):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (the library has no CPU path)")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"{name} must have dtype {dtype}, got {t.dtype}")
    return ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream: Optional[torch.cuda.Stream]):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def build_workspace_bytes(V: int, D: int, k: int) -> int:
    return int(load_library().lantern_build_workspace_bytes(V, D, k))


METRICS = {"l2": 0, "cosine": 1}
DIVERGENCES = {"tvd": 0, "jsd": 1}


def build_neighbors(codebook: torch.Tensor, k: int, *, with_dist: bool = True, metric: str = "l2",
                    workspace: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """lantern_build_neighbors[_metric]: [V, D] fp32 codebook -> (idx [V, k] int32, dist [V, k] fp32 or None).
    metric "l2" (squared l2 distances) or "cosine" (dist = 2 - 2 cos on unit-length codes)."""
    lib = load_library()
    V, D = codebook.shape
    if metric not in METRICS:
        raise ValueError(f"metric must be one of {sorted(METRICS)}")
    with torch.cuda.device(codebook.device):
        idx = torch.empty((V, k), dtype=torch.int32, device=codebook.device)
        dist = torch.empty((V, k), dtype=torch.float32, device=codebook.device) if with_dist else None
        need = int(lib.lantern_build_workspace_bytes_metric(V, D, int(k), METRICS[metric]))
        if workspace is None and need:
            workspace = torch.empty(need, dtype=torch.uint8, device=codebook.device)
        rc = lib.lantern_build_neighbors_metric(
            _ptr(codebook, torch.float32, "codebook"), V, D, int(k), METRICS[metric], _ptr(idx), _ptr(dist),
            _ptr(workspace), workspace.numel() if workspace is not None else 0, _stream_ptr(stream))
    if rc != 0:
        raise LanternError(rc, "lantern_build_neighbors_metric")
    return idx, dist


def verify_workspace_bytes(B: int, N: int, V: int = 16384, k: int = 1, dtype: int = BF16, top_k: int = 0) -> int:
    """lantern_verify_workspace_bytes_ex: scratch bytes of one verify() call (0 for a refused shape)."""
    return int(load_library().lantern_verify_workspace_bytes_ex(B, N, V, k, dtype, int(top_k)))


E_DATA = -6


def last_status(workspace: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> int:
    """lantern_last_status: OR of the status bits of every sequence of the last verify() call that used
    `workspace` (0 = none); waits for the stream."""
    bits = ctypes.c_int32(0)
    with torch.cuda.device(workspace.device):
        rc = load_library().lantern_last_status(_ptr(workspace), _stream_ptr(stream), ctypes.byref(bits))
    if rc not in (0, E_DATA):
        raise LanternError(rc, "lantern_last_status")
    return int(bits.value)


def verify_counts(workspace: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> dict:
    """lantern_verify_counts: work accounting of the last verify() call that used `workspace`."""
    out = (ctypes.c_int64 * 6)()
    with torch.cuda.device(workspace.device):
        rc = load_library().lantern_verify_counts(_ptr(workspace), _stream_ptr(stream), out)
    if rc != 0:
        raise LanternError(rc, "lantern_verify_counts")
    return dict(contexts=int(out[0]), evaluated=int(out[1]), skipped=int(out[2]), from_q=int(out[3]),
                nodes_tested=int(out[4]), slow_topk_rows=int(out[5]))


def debug_wait_test(max_tries: int = 0, withhold_context: int = -1) -> None:
    """lantern_debug_wait_test: self-test hook of the bounded waits (0, -1 restores the defaults)."""
    rc = load_library().lantern_debug_wait_test(int(max_tries), int(withhold_context))
    if rc != 0:
        raise LanternError(rc, "lantern_debug_wait_test")


@dataclasses.dataclass
class VerifyOutputs:
    accept_len: torch.Tensor            # [B] int32
    next_token: torch.Tensor            # [B] int32
    accept_path: Optional[torch.Tensor]  # [B, N] int32
    status: Optional[torch.Tensor]      # [B] int32
    node_qa: Optional[torch.Tensor]     # [B, N] fp32
    node_px: Optional[torch.Tensor]     # [B, N] fp32
    node_m: Optional[torch.Tensor]      # [B, N] int32


def verify(target_logits: torch.Tensor, draft_logits: Optional[torch.Tensor], cfg_scale: float, T: float,
           draft_tokens: Optional[torch.Tensor], tree_parents: Optional[torch.Tensor], neighbor_idx: torch.Tensor,
           delta: float, uniforms: Optional[torch.Tensor], *, out: Optional[VerifyOutputs] = None, trace: bool = False,
           workspace: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None,
           divergence: str = "tvd", top_k: int = 0) -> VerifyOutputs:
    """lantern_verify_ex on torch tensors (divergence "tvd" and top_k = 0 are lantern_verify).

    target_logits [C, B, N+1, V] (C = 2: conditional, unconditional; C = 1: no guidance), fp32 or bf16;
    draft_logits [B, N+1, V]; draft_tokens / tree_parents [B, N] int32 (tree_parents None = chain);
    neighbor_idx [V, k] int32; uniforms [B, N+1] fp32.  Outputs are allocated unless `out` is given.
    T == 0 selects greedy decoding: draft_logits and uniforms are not read and may be None.
    divergence "tvd" | "jsd": what delta bounds (Section 5.3.2); top_k: logit filter, 0 = off (Appendix B.2).
    """
    if divergence not in DIVERGENCES:
        raise ValueError(f"divergence must be one of {sorted(DIVERGENCES)}")
    lib = load_library()
    if T != 0 and (uniforms is None or (draft_logits is None and target_logits.shape[2] > 1)):
        raise ValueError("sampling (T > 0) needs draft_logits and uniforms")
    C, B, R, V = target_logits.shape
    N = R - 1
    if C not in (1, 2):
        raise ValueError("target_logits must have 1 or 2 guidance branches")
    if target_logits.dtype == torch.bfloat16:
        dtype = BF16
    elif target_logits.dtype == torch.float32:
        dtype = F32
    else:
        raise ValueError("logits must be float32 or bfloat16")
    dev = target_logits.device
    k = neighbor_idx.shape[1]
    if neighbor_idx.shape[0] != V:
        raise ValueError("neighbor_idx must have V rows")
    with torch.cuda.device(dev):
        if out is None:
            i32 = dict(dtype=torch.int32, device=dev)
            out = VerifyOutputs(
                accept_len=torch.empty(B, **i32), next_token=torch.empty(B, **i32),
                accept_path=torch.empty((B, N), **i32), status=torch.empty(B, **i32),
                node_qa=torch.empty((B, N), dtype=torch.float32, device=dev) if trace else None,
                node_px=torch.empty((B, N), dtype=torch.float32, device=dev) if trace else None,
                node_m=torch.empty((B, N), **i32) if trace else None)
        need = verify_workspace_bytes(B, N, V, int(k), dtype, top_k)
        if workspace is None:
            workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
        rc = lib.lantern_verify_ex(
            _ptr(target_logits, None, "target_logits"), _ptr(draft_logits, target_logits.dtype, "draft_logits"),
            dtype, float(cfg_scale), int(C == 2), float(T), _ptr(draft_tokens, torch.int32, "draft_tokens"),
            _ptr(tree_parents, torch.int32, "tree_parents"), _ptr(neighbor_idx, torch.int32, "neighbor_idx"),
            int(k), float(delta), DIVERGENCES[divergence], int(top_k), _ptr(uniforms, torch.float32, "uniforms"),
            B, N, V, _ptr(out.accept_len, torch.int32), _ptr(out.next_token, torch.int32),
            _ptr(out.accept_path, torch.int32), _ptr(out.status, torch.int32), _ptr(out.node_qa, torch.float32),
            _ptr(out.node_px, torch.float32), _ptr(out.node_m, torch.int32), _ptr(workspace),
            workspace.numel(), _stream_ptr(stream))
    if rc != 0:
        raise LanternError(rc, "lantern_verify_ex")
    return out


def aggregate_all(logits: torch.Tensor, cfg_scale: float, T: float, neighbor_idx: torch.Tensor, delta: float, *,
                  with_m: bool = True, stream: Optional[torch.cuda.Stream] = None):
    """lantern_aggregate_all: logits [C, rows, V] -> (agg [rows, V] fp32, m [rows, V] int32 or None, status [rows]).
    A benchmark of the V x k gather-sum (the mass of A_{k,delta}(x) for every token x); verify() does not use it."""
    lib = load_library()
    C, rows, V = logits.shape
    if C not in (1, 2):
        raise ValueError("logits must have 1 or 2 guidance branches")
    dtype = BF16 if logits.dtype == torch.bfloat16 else F32
    if logits.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("logits must be float32 or bfloat16")
    dev = logits.device
    with torch.cuda.device(dev):
        agg = torch.empty((rows, V), dtype=torch.float32, device=dev)
        m = torch.empty((rows, V), dtype=torch.int32, device=dev) if with_m else None
        status = torch.empty(rows, dtype=torch.int32, device=dev)
        rc = lib.lantern_aggregate_all(_ptr(logits, None, "logits"), dtype, float(cfg_scale), int(C == 2), float(T),
                                       _ptr(neighbor_idx, torch.int32, "neighbor_idx"), int(neighbor_idx.shape[1]),
                                       float(delta), rows, V, _ptr(agg), _ptr(m), _ptr(status), _stream_ptr(stream))
    if rc != 0:
        raise LanternError(rc, "lantern_aggregate_all")
    return agg, m, status


def verify_launch_count(greedy: bool = False, top_k_active: bool = False) -> int:
    """Stream operations (kernels + 1 memset) enqueued by one verify() call."""
    return int(load_library().lantern_verify_launch_count(int(greedy), int(top_k_active)))


def profile_events(before: Optional[torch.cuda.Event], after: Optional[torch.cuda.Event]) -> None:
    """lantern_verify_profile_events: record `before` / `after` around the fused context kernel of every
    later verify() call of this thread (both None switches it off).  Events need enable_timing=True and
    must have been recorded once (torch creates the CUDA event lazily)."""
    lib = load_library()
    if before is None or after is None:
        rc = lib.lantern_verify_profile_events(None, None)
    else:
        rc = lib.lantern_verify_profile_events(ctypes.c_void_p(before.cuda_event), ctypes.c_void_p(after.cuda_event))
    if rc != 0:
        raise LanternError(rc, "lantern_verify_profile_events")


STATIC_WORKSPACE_BYTES = 6 << 20


def verify_static(target_logits: torch.Tensor, draft_logits: Optional[torch.Tensor], cfg_scale: float, T: float,
                  draft_tokens: Optional[torch.Tensor], tree_parents: Optional[torch.Tensor],
                  neighbor_idx: torch.Tensor, delta: float, uniforms: Optional[torch.Tensor], *, out: VerifyOutputs,
                  stream: Optional[torch.cuda.Stream] = None) -> VerifyOutputs:
    """lantern_verify_static: verify() for callers that must not allocate device memory.

    The library's scratch comes from a fixed 6 MiB array inside its device image, so nothing is
    allocated here either: the caller passes every output tensor in `out` (allocated whenever it was
    still allowed to).  The call is refused (LanternError, code -4) if verify_workspace_bytes(B, N, V, k)
    exceeds STATIC_WORKSPACE_BYTES.  Calls on one device share the array: do not let two of them run
    on the GPU at the same time.  Make the first call on a device outside stream capture."""
    lib = load_library()
    C, B, R, V = target_logits.shape
    N = R - 1
    if C not in (1, 2):
        raise ValueError("target_logits must have 1 or 2 guidance branches")
    if target_logits.dtype == torch.bfloat16:
        dtype = BF16
    elif target_logits.dtype == torch.float32:
        dtype = F32
    else:
        raise ValueError("logits must be float32 or bfloat16")
    if neighbor_idx.shape[0] != V:
        raise ValueError("neighbor_idx must have V rows")
    with torch.cuda.device(target_logits.device):
        rc = lib.lantern_verify_static(
            _ptr(target_logits, None, "target_logits"), _ptr(draft_logits, target_logits.dtype, "draft_logits"),
            dtype, float(cfg_scale), int(C == 2), float(T), _ptr(draft_tokens, torch.int32, "draft_tokens"),
            _ptr(tree_parents, torch.int32, "tree_parents"), _ptr(neighbor_idx, torch.int32, "neighbor_idx"),
            int(neighbor_idx.shape[1]), float(delta), _ptr(uniforms, torch.float32, "uniforms"), B, N, V,
            _ptr(out.accept_len, torch.int32), _ptr(out.next_token, torch.int32),
            _ptr(out.accept_path, torch.int32), _ptr(out.status, torch.int32), _ptr(out.node_qa, torch.float32),
            _ptr(out.node_px, torch.float32), _ptr(out.node_m, torch.int32), _stream_ptr(stream))
    if rc != 0:
        raise LanternError(rc, "lantern_verify_static")
    return out


def kernel_revision() -> int:
    """Revision number of the fused verification kernel (matches stored profiler counters to code)."""
    return int(load_library().lantern_kernel_revision())
