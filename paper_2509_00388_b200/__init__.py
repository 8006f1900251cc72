"""GraphKV prefill KV-cache compression on B200 (sm_100a): CUDA kernels behind a C ABI.

`workloads` draws the seeded synthetic inputs; `binding` is the thin ctypes layer over
libgraphkv.so (built from csrc/ by `build`).  Nothing here computes on the CPU: the
binding raises if the CUDA library is missing.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads"]
