"""ctypes binding of libgraphkv.so: argument marshalling only.

Every function takes CUDA torch tensors, fills a `graphkv_params` struct from their shapes and
strides, and passes raw device pointers plus the current CUDA stream to the C entry point of
the same name (declared in include/graphkv.h).  No step of the path runs here, and there is no
CPU route: loading fails loudly if the CUDA library has not been built.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Tuple

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("GRAPHKV_LIB") or os.path.join(HERE, "libgraphkv.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_BUILTIN_SCRATCH = range(7)
BUILTIN_SCRATCH_BYTES = 16 << 20
BF16, F32 = 0, 1
POOL_MAX, POOL_AVG = 0, 1
SIGNAL_DECAY, SIGNAL_ENHANCE, SIGNAL_EVICT = 0, 1, 2
TENSOR_K, TENSOR_V = 0, 1

EXPORTS = ("graphkv_workspace_bytes", "graphkv_resolve_neighbors", "graphkv_score",
           "graphkv_propagate", "graphkv_select_gather", "graphkv_compress",
           "graphkv_read_status", "graphkv_status_string", "graphkv_launch_count",
           "graphkv_trace_enable", "graphkv_trace_read", "graphkv_builtin_scratch_needed",
           "graphkv_score_noalloc", "graphkv_read_status_noalloc", "graphkv_read_neighbors", "graphkv_phase_timing_read", "graphkv_score_knorm",
           "graphkv_propagate_edges", "graphkv_compress_layers", "graphkv_decode_workspace_bytes",
           "graphkv_decode_attention")


class GraphKVError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


class Params(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("seq_len", C.c_int32), ("window", C.c_int32),
                ("budget", C.c_int32), ("pool_kernel", C.c_int32), ("pool_mode", C.c_int32),
                ("topk_nodes", C.c_int32), ("neighbors", C.c_int32), ("rounds", C.c_int32),
                ("decay", C.c_float), ("dtype", C.c_int32),
                ("q_stride", C.c_int64 * 3), ("k_stride", C.c_int64 * 3),
                ("v_stride", C.c_int64 * 3), ("signal", C.c_int32), ("reselect", C.c_int32)]


class TraceRecord(C.Structure):
    _fields_ = [("name", C.c_char * 40), ("ms", C.c_float)]


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    """The loaded CUDA library.  Raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2509_00388_b200.build` "
                "(nvcc, sm_100a).  This library has no CPU or PyTorch fallback.")
        L = C.CDLL(LIB_PATH)
        P = C.POINTER(Params)
        vp, sz = C.c_void_p, C.c_size_t
        L.graphkv_workspace_bytes.restype = sz
        L.graphkv_workspace_bytes.argtypes = [P]
        L.graphkv_resolve_neighbors.restype = C.c_int32
        L.graphkv_resolve_neighbors.argtypes = [C.c_int32, C.c_int32]
        L.graphkv_score.restype = C.c_int
        L.graphkv_score.argtypes = [P, vp, vp, vp, vp, sz, vp]
        L.graphkv_propagate.restype = C.c_int
        L.graphkv_propagate.argtypes = [P, vp, vp, vp, vp, sz, vp]
        L.graphkv_select_gather.restype = C.c_int
        L.graphkv_select_gather.argtypes = [P, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.graphkv_compress.restype = C.c_int
        L.graphkv_compress.argtypes = [P, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.graphkv_compress_layers.restype = C.c_int
        L.graphkv_compress_layers.argtypes = [P, C.POINTER(C.c_int32), vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.graphkv_decode_workspace_bytes.restype = sz
        L.graphkv_decode_workspace_bytes.argtypes = [P]
        L.graphkv_decode_attention.restype = C.c_int
        L.graphkv_decode_attention.argtypes = [P, vp, vp, vp, vp, vp, sz, vp]
        L.graphkv_read_status.restype = C.c_int
        L.graphkv_read_status.argtypes = [vp, vp]
        L.graphkv_score_knorm.restype = C.c_int
        L.graphkv_score_knorm.argtypes = [P, vp, vp, vp]
        L.graphkv_propagate_edges.restype = C.c_int
        L.graphkv_propagate_edges.argtypes = [P, vp, vp, C.c_int32, C.c_int32, vp, vp, vp, sz, vp]
        L.graphkv_read_neighbors.restype = C.c_int
        L.graphkv_read_neighbors.argtypes = [P, vp, sz, vp, vp, vp]
        L.graphkv_phase_timing_read.restype = C.c_int32
        L.graphkv_phase_timing_read.argtypes = [C.POINTER(C.c_uint64)]
        L.graphkv_builtin_scratch_needed.restype = sz
        L.graphkv_builtin_scratch_needed.argtypes = [P]
        L.graphkv_score_noalloc.restype = C.c_int
        L.graphkv_score_noalloc.argtypes = [P, vp, vp, vp, vp]
        L.graphkv_read_status_noalloc.restype = C.c_int
        L.graphkv_read_status_noalloc.argtypes = [vp]
        L.graphkv_status_string.restype = C.c_char_p
        L.graphkv_status_string.argtypes = [C.c_int]
        L.graphkv_launch_count.restype = C.c_int64
        L.graphkv_launch_count.argtypes = []
        L.graphkv_trace_enable.restype = None
        L.graphkv_trace_enable.argtypes = [C.c_int32]
        L.graphkv_trace_read.restype = C.c_int32
        L.graphkv_trace_read.argtypes = [C.POINTER(TraceRecord), C.c_int32]
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().graphkv_status_string(int(code)).decode()


def resolve_neighbors(n_prefix: int, neighbors: int) -> int:
    return int(lib().graphkv_resolve_neighbors(n_prefix, neighbors))


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise TypeError(f"unsupported dtype {t.dtype}")


def _strides3(t: Optional[torch.Tensor]):
    if t is None:
        return (C.c_int64 * 3)(0, 0, 128)
    assert t.dim() == 4 and t.stride(3) == 1, "expected [batch, heads, rows, D] with D contiguous"
    return (C.c_int64 * 3)(t.stride(0), t.stride(1), t.stride(2))


def make_params(K: torch.Tensor, *, window: int, n_q_heads: Optional[int] = None,
                Qw: Optional[torch.Tensor] = None, V: Optional[torch.Tensor] = None,
                budget: int = 1, pool_kernel: int = 1, topk_nodes: int = 0, neighbors: int = 0,
                rounds: int = 0, decay: float = 1.0, pool_mode: int = 0, signal: int = 0,
                reselect: int = 0) -> Params:
    b, hkv, ell, d = K.shape
    hq = Qw.shape[1] if Qw is not None else (n_q_heads or hkv)
    p = Params()
    p.batch, p.n_q_heads, p.n_kv_heads, p.head_dim = b, hq, hkv, d
    p.seq_len, p.window, p.budget = ell, window, budget
    p.pool_kernel, p.pool_mode = pool_kernel, pool_mode
    p.signal, p.reselect = signal, reselect
    p.topk_nodes, p.neighbors, p.rounds, p.decay = topk_nodes, neighbors, rounds, decay
    p.dtype = _dtype_code(K)
    p.q_stride = _strides3(Qw)
    p.k_stride = _strides3(K)
    p.v_stride = _strides3(V if V is not None else K)
    return p


def workspace_bytes(p: Params) -> int:
    return int(lib().graphkv_workspace_bytes(C.byref(p)))


def alloc_workspace(p: Params, device) -> torch.Tensor:
    n = workspace_bytes(p)
    if n == 0:
        raise GraphKVError(ERR_INVALID_ARG, "graphkv_workspace_bytes")
    # zero-filled: the status word at its head is only cleared by the scoring calls
    return torch.zeros(n, dtype=torch.uint8, device=device)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(device) -> int:
    return torch.cuda.current_stream(device).cuda_stream


def _check(code: int, where: str) -> None:
    if code != OK:
        raise GraphKVError(code, where)


def graphkv_score(p: Params, Qw: torch.Tensor, K: torch.Tensor, scores: torch.Tensor,
                  ws: torch.Tensor) -> None:
    _check(lib().graphkv_score(C.byref(p), _ptr(Qw), _ptr(K), _ptr(scores), _ptr(ws),
                               ws.numel(), _stream(K.device)), "graphkv_score")


def builtin_scratch_needed(p: Params) -> int:
    return int(lib().graphkv_builtin_scratch_needed(C.byref(p)))


def graphkv_score_noalloc(p: Params, Qw: torch.Tensor, K: torch.Tensor, scores: torch.Tensor) -> None:
    """graphkv_score without a workspace: the scratch is the library's built-in device array, so
    the call allocates nothing (for callers inside regions where device allocation is closed).
    Raises GraphKVError(ERR_BUILTIN_SCRATCH) when the problem does not fit that array."""
    _check(lib().graphkv_score_noalloc(C.byref(p), _ptr(Qw), _ptr(K), _ptr(scores),
                                       _stream(K.device)), "graphkv_score_noalloc")


def graphkv_read_status_noalloc(device) -> int:
    return int(lib().graphkv_read_status_noalloc(_stream(device)))


def graphkv_propagate(p: Params, K: torch.Tensor, scores: torch.Tensor,
                      src_idx_out: Optional[torch.Tensor], ws: torch.Tensor) -> None:
    _check(lib().graphkv_propagate(C.byref(p), _ptr(K), _ptr(scores), _ptr(src_idx_out),
                                   _ptr(ws), ws.numel(), _stream(K.device)),
           "graphkv_propagate")


def graphkv_score_knorm(p: Params, K: torch.Tensor, scores: torch.Tensor) -> None:
    _check(lib().graphkv_score_knorm(C.byref(p), _ptr(K), _ptr(scores), _stream(K.device)),
           "graphkv_score_knorm")


def graphkv_propagate_edges(p: Params, K: Optional[torch.Tensor], V: Optional[torch.Tensor],
                            src_tensor: int, all_tensor: int, scores: torch.Tensor,
                            src_idx_out: Optional[torch.Tensor], ws: torch.Tensor) -> None:
    _check(lib().graphkv_propagate_edges(C.byref(p), _ptr(K), _ptr(V), src_tensor, all_tensor,
                                         _ptr(scores), _ptr(src_idx_out), _ptr(ws), ws.numel(),
                                         _stream(scores.device)), "graphkv_propagate_edges")


def graphkv_select_gather(p: Params, scores: torch.Tensor, K: Optional[torch.Tensor],
                          V: Optional[torch.Tensor], K_out: Optional[torch.Tensor],
                          V_out: Optional[torch.Tensor], idx_out: torch.Tensor,
                          ws: torch.Tensor) -> None:
    _check(lib().graphkv_select_gather(C.byref(p), _ptr(scores), _ptr(K), _ptr(V), _ptr(K_out),
                                       _ptr(V_out), _ptr(idx_out), _ptr(ws), ws.numel(),
                                       _stream(scores.device)), "graphkv_select_gather")


def graphkv_compress(p: Params, Qw: torch.Tensor, K: torch.Tensor, V: torch.Tensor,
                     K_out: torch.Tensor, V_out: torch.Tensor, idx_out: torch.Tensor,
                     scores_out: Optional[torch.Tensor], ws: torch.Tensor) -> None:
    _check(lib().graphkv_compress(C.byref(p), _ptr(Qw), _ptr(K), _ptr(V), _ptr(K_out),
                                  _ptr(V_out), _ptr(idx_out), _ptr(scores_out), _ptr(ws),
                                  ws.numel(), _stream(K.device)), "graphkv_compress")


def graphkv_compress_layers(p: Params, budgets, Qw: torch.Tensor, K: torch.Tensor, V: torch.Tensor,
                            K_out: torch.Tensor, V_out: torch.Tensor, idx_out: torch.Tensor,
                            scores_out: Optional[torch.Tensor], ws: torch.Tensor) -> None:
    """graphkv_compress with a budget per batch element (layer); p.budget is the outputs' capacity."""
    arr = (C.c_int32 * p.batch)(*[int(b) for b in budgets])
    _check(lib().graphkv_compress_layers(C.byref(p), arr, _ptr(Qw), _ptr(K), _ptr(V), _ptr(K_out),
                                         _ptr(V_out), _ptr(idx_out), _ptr(scores_out), _ptr(ws),
                                         ws.numel(), _stream(K.device)), "graphkv_compress_layers")


def decode_params(q: torch.Tensor, K: torch.Tensor, V: torch.Tensor) -> Params:
    """Params of a decoding step: q [batch, n_q_heads, D], K and V [batch, n_kv_heads, rows, D]."""
    p = Params()
    p.batch, p.n_q_heads, p.n_kv_heads, p.head_dim = K.shape[0], q.shape[1], K.shape[1], K.shape[3]
    p.seq_len, p.window, p.budget, p.pool_kernel = K.shape[2], 1, 1, 1
    p.dtype = _dtype_code(K)
    p.q_stride = (C.c_int64 * 3)(q.stride(0), q.stride(1), K.shape[3])
    p.k_stride = _strides3(K)
    p.v_stride = _strides3(V)
    return p


def graphkv_decode_attention(p: Params, q: torch.Tensor, K: torch.Tensor, V: torch.Tensor,
                             out: torch.Tensor, ws: torch.Tensor) -> None:
    _check(lib().graphkv_decode_attention(C.byref(p), _ptr(q), _ptr(K), _ptr(V), _ptr(out), _ptr(ws),
                                          ws.numel(), _stream(K.device)), "graphkv_decode_attention")


def decode_workspace(p: Params, device) -> torch.Tensor:
    n = int(lib().graphkv_decode_workspace_bytes(C.byref(p)))
    if n == 0:
        raise GraphKVError(ERR_INVALID_ARG, "graphkv_decode_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def graphkv_read_status(ws: torch.Tensor) -> int:
    return int(lib().graphkv_read_status(_ptr(ws), _stream(ws.device)))


def graphkv_read_neighbors(p: Params, ws: torch.Tensor, nbr_idx_out: Optional[torch.Tensor],
                           nbr_e_out: Optional[torch.Tensor]) -> None:
    _check(lib().graphkv_read_neighbors(C.byref(p), _ptr(ws), ws.numel(), _ptr(nbr_idx_out),
                                        _ptr(nbr_e_out), _stream(ws.device)),
           "graphkv_read_neighbors")


def graphkv_launch_count() -> int:
    return int(lib().graphkv_launch_count())


def graphkv_trace_enable(enable: bool) -> None:
    lib().graphkv_trace_enable(1 if enable else 0)


def graphkv_trace_read(capacity: int = 1 << 16):
    """[(kernel name, device ms), ...] of the launches traced since the last read."""
    buf = (TraceRecord * capacity)()
    n = lib().graphkv_trace_read(buf, capacity)
    return [(buf[i].name.decode(), float(buf[i].ms)) for i in range(n)]


def graphkv_phase_timing_read():
    """Per-kernel phase times of a library built with GRAPHKV_PHASE_TIMING, or None.
    Returns {kernel index: (CTAs, [(mean ns, max ns) per phase])}; phase 0 is the whole CTA."""
    n_k, n_s = 8, 24
    buf = (C.c_uint64 * (n_k * n_s * 2 + n_k))()
    if not lib().graphkv_phase_timing_read(buf):
        return None
    out = {}
    for k in range(n_k):
        cnt = buf[n_k * n_s * 2 + k]
        if cnt:
            out[k] = (int(cnt), [(buf[(k * n_s + i) * 2] / cnt, int(buf[(k * n_s + i) * 2 + 1]))
                                 for i in range(n_s)])
    return out


def alloc_outputs(p: Params, like: torch.Tensor, want_scores: bool = True
                  ) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor, Optional[torch.Tensor]]:
    """Dense output tensors of the shapes the C ABI writes."""
    n = p.seq_len - p.window
    shape = (p.batch, p.n_kv_heads, p.budget + p.window, p.head_dim)
    K_out = torch.empty(shape, dtype=like.dtype, device=like.device)
    V_out = torch.empty(shape, dtype=like.dtype, device=like.device)
    idx = torch.empty((p.batch, p.n_kv_heads, p.budget), dtype=torch.int32, device=like.device)
    s = (torch.empty((p.batch, p.n_kv_heads, n), dtype=torch.float32, device=like.device)
         if want_scores else None)
    return K_out, V_out, idx, s
