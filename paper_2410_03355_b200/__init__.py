"""LANTERN relaxed speculative verification for B200 (sm_100a).

Thin Python binding over the C ABI declared in include/lantern.h.  Every step of the method
runs in the CUDA library; this package only marshals torch tensors into pointers.
"""
from .binding import (BF16, F32, LanternError, kernel_revision, build_neighbors, build_workspace_bytes, library_path,
                      load_library, profile_events, status_string, verify, verify_launch_count,
                      verify_static, verify_workspace_bytes, VerifyOutputs, STATIC_WORKSPACE_BYTES,
                      ST_BAD_TOKEN, ST_BAD_PARENT, ST_BAD_UNIFORM, ST_NONFINITE, ST_DEGENERATE, ST_BAD_TABLE,
                      ST_INTERNAL, METRICS, DIVERGENCES, aggregate_all, last_status, verify_counts,
                      debug_wait_test)

__all__ = ["BF16", "F32", "LanternError", "kernel_revision", "build_neighbors", "build_workspace_bytes", "library_path",
           "load_library", "profile_events", "status_string", "verify", "verify_launch_count", "verify_static", "verify_workspace_bytes", "VerifyOutputs", "STATIC_WORKSPACE_BYTES",
           "ST_BAD_TOKEN", "ST_BAD_PARENT", "ST_BAD_UNIFORM", "ST_NONFINITE", "ST_DEGENERATE", "ST_BAD_TABLE",
           "ST_INTERNAL", "METRICS", "DIVERGENCES", "aggregate_all", "last_status", "verify_counts", "debug_wait_test"]
