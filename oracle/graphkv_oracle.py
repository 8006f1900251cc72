"""ctypes front end of the C oracle (oracle/graphkv_oracle.c).

Test infrastructure: only tests, the smoke check and the benchmark's cpu-baseline leg import
this.  Inputs are CPU torch tensors; bf16 inputs are widened to fp32 (exact) for the
arithmetic and passed as raw bytes for the gather.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass
from typing import Optional, Tuple

import numpy as np
import torch

from . import build as _build


class _Params(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("seq_len", C.c_int32), ("window", C.c_int32),
                ("budget", C.c_int32), ("pool_kernel", C.c_int32), ("topk_nodes", C.c_int32),
                ("neighbors", C.c_int32), ("rounds", C.c_int32), ("decay", C.c_double),
                ("pool_mode", C.c_int32), ("signal", C.c_int32), ("reselect", C.c_int32)]


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.okv_resolve_neighbors.restype = C.c_int32
        _lib.okv_num_threads.restype = C.c_int32
        for name in ("okv_topk", "okv_score_unit", "okv_score_knorm_unit", "okv_edges2_unit",
                     "okv_decode_attention_unit",
                     "okv_propagate2_unit", "okv_propagate_reselect_unit", "okv_edges_unit", "okv_propagate_unit",
                     "okv_select_unit", "okv_gather_unit", "okv_score", "okv_propagate",
                     "okv_select_gather", "okv_compress"):
            getattr(_lib, name).restype = None
    return _lib


def num_threads() -> int:
    return int(lib().okv_num_threads())


def resolve_neighbors(n_prefix: int, neighbors: int) -> int:
    return int(lib().okv_resolve_neighbors(C.c_int32(n_prefix), C.c_int32(neighbors)))


def _f32(t: torch.Tensor) -> np.ndarray:
    return np.ascontiguousarray(t.detach().cpu().to(torch.float32).numpy())


def _raw(t: torch.Tensor) -> Tuple[np.ndarray, int]:
    t = t.detach().cpu().contiguous()
    return t.view(torch.uint8).numpy().reshape(-1), t.element_size()


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


@dataclass
class Shape:
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    seq_len: int
    window: int

    @property
    def n_prefix(self) -> int:
        return self.seq_len - self.window


def _shape(Qw: Optional[torch.Tensor], K: torch.Tensor, window: int,
           n_q_heads: Optional[int] = None) -> Shape:
    b, hkv, ell, d = K.shape
    hq = Qw.shape[1] if Qw is not None else (n_q_heads or hkv)
    if Qw is not None:
        assert Qw.shape == (b, hq, window, d), "Qw must be [batch, n_q_heads, W, D]"
    assert hq % hkv == 0 and 1 <= window < ell
    return Shape(b, hq, hkv, d, ell, window)


POOL_MAX, POOL_AVG = 0, 1
SIGNAL_DECAY, SIGNAL_ENHANCE, SIGNAL_EVICT = 0, 1, 2


def _params(sh: Shape, budget=1, pool_kernel=1, topk_nodes=0, neighbors=0, rounds=0,
            decay=1.0, pool_mode=0, signal=0, reselect=0) -> _Params:
    n = sh.n_prefix
    assert pool_kernel >= 1 and pool_kernel % 2 == 1
    assert 1 <= budget <= n and 0 <= topk_nodes <= n and rounds >= 0
    assert 0 <= neighbors <= n - 1
    return _Params(sh.batch, sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.seq_len, sh.window,
                   budget, pool_kernel, topk_nodes, neighbors, rounds, float(decay),
                   int(pool_mode), int(signal), int(reselect))


def score(Qw: torch.Tensor, K: torch.Tensor, window: int, pool_kernel: int,
          pool_mode: int = 0) -> torch.Tensor:
    """Pooled SnapKV-style scores, fp32 [batch, n_kv_heads, N]."""
    sh = _shape(Qw, K, window)
    p = _params(sh, pool_kernel=pool_kernel, pool_mode=pool_mode)
    q, k = _f32(Qw), _f32(K)
    s = np.empty((sh.batch, sh.n_kv_heads, sh.n_prefix), dtype=np.float32)
    lib().okv_score(C.byref(p), _ptr(q), _ptr(k), _ptr(s))
    return torch.from_numpy(s)


def score_unit(Qg: torch.Tensor, Kh: torch.Tensor, pool_kernel: int, pool_mode: int = 0
               ) -> Tuple[torch.Tensor, torch.Tensor]:
    """One KV head: Qg [G, W, D], Kh [L, D] -> (unpooled mass fp64 [N], pooled score fp32 [N])."""
    g, w, d = Qg.shape
    n = Kh.shape[0] - w
    q, k = _f32(Qg), _f32(Kh)
    a = np.empty(n, dtype=np.float64)
    s = np.empty(n, dtype=np.float32)
    lib().okv_score_unit(_ptr(q), _ptr(k), C.c_int32(g), C.c_int32(w), C.c_int32(d),
                         C.c_int32(n), C.c_int32(pool_kernel), C.c_int32(pool_mode), _ptr(a), _ptr(s))
    return torch.from_numpy(a), torch.from_numpy(s)


def score_knorm(K: torch.Tensor, window: int) -> torch.Tensor:
    """KNorm initial scores 1 / ||k_j|| of the prefix keys, fp32 [batch, n_kv_heads, N]."""
    b, hkv, ell, d = K.shape
    n = ell - window
    k = _f32(K)
    s = np.empty((b, hkv, n), dtype=np.float32)
    for bi in range(b):
        for h in range(hkv):
            kh = np.ascontiguousarray(k[bi, h])
            lib().okv_score_knorm_unit(_ptr(kh), C.c_int32(n), C.c_int32(d), _ptr(s[bi, h]))
    return torch.from_numpy(s)


def decode_attention(q: torch.Tensor, K: torch.Tensor, V: torch.Tensor) -> torch.Tensor:
    """One decoding step's attention over a cache: q [batch, n_q_heads, D], K and V
    [batch, n_kv_heads, rows, D] -> fp64 [batch, n_q_heads, D]."""
    b, hkv, rows, d = K.shape
    g = q.shape[1] // hkv
    qf, kf, vf = _f32(q), _f32(K), _f32(V)
    out = np.empty((b, q.shape[1], d), dtype=np.float64)
    for bi in range(b):
        for h in range(hkv):
            qq = np.ascontiguousarray(qf[bi, h * g:(h + 1) * g])
            kk, vv = np.ascontiguousarray(kf[bi, h]), np.ascontiguousarray(vf[bi, h])
            oo = np.empty((g, d), dtype=np.float64)
            lib().okv_decode_attention_unit(_ptr(qq), _ptr(kk), _ptr(vv), C.c_int32(g), C.c_int32(rows),
                                            C.c_int32(d), _ptr(oo))
            out[bi, h * g:(h + 1) * g] = oo
    return torch.from_numpy(out)


def edges_unit(Kh: torch.Tensor, n_prefix: int, i: int,
               Sh: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Eq. 1 for source i against every prefix key of one head; fp64 [N] (entry i included).
    With Sh the source's vector is row i of Sh instead (other edge kinds)."""
    k = _f32(Kh)
    sv = k if Sh is None else _f32(Sh)
    e = np.empty(n_prefix, dtype=np.float64)
    lib().okv_edges2_unit(_ptr(sv), _ptr(k), C.c_int32(n_prefix), C.c_int32(k.shape[1]), C.c_int32(i),
                          _ptr(e))
    return torch.from_numpy(e)


def topk(x: torch.Tensor, k: int, skip: int = -1) -> torch.Tensor:
    """Indices of the k largest entries of a 1-D fp32 row, (value desc, index asc) order."""
    xv = np.ascontiguousarray(x.detach().cpu().numpy(), dtype=np.float32)
    out = np.empty(k, dtype=np.int32)
    lib().okv_topk(_ptr(xv), C.c_int32(xv.shape[0]), C.c_int32(k), C.c_int32(skip), _ptr(out))
    return torch.from_numpy(out)


def propagate_unit(Kh: torch.Tensor, scores: torch.Tensor, n_prefix: int, topk_nodes: int,
                   neighbors: int, rounds: int, decay: float,
                   forced_src: Optional[torch.Tensor] = None,
                   forced_nbr: Optional[torch.Tensor] = None, signal: int = 0,
                   Sh: Optional[torch.Tensor] = None):
    """One KV head with optional teacher forcing.  Returns (scores fp32 [N], src [K_src],
    nbr [K_src, m], nbr_e fp64 [K_src, m]).  Sh: tensor the sources' vectors come from (default
    the same as the swept one)."""
    k = _f32(Kh)
    sv = k if Sh is None else _f32(Sh)
    m = resolve_neighbors(n_prefix, neighbors)
    s = np.array(scores.detach().cpu().numpy(), dtype=np.float32, copy=True)
    src = np.zeros(max(topk_nodes, 1), dtype=np.int32)
    nbr = np.zeros((max(topk_nodes, 1), m), dtype=np.int32)
    nbr_e = np.zeros((max(topk_nodes, 1), m), dtype=np.float64)
    fs = None if forced_src is None else np.ascontiguousarray(
        forced_src.detach().cpu().numpy(), dtype=np.int32)
    fn = None if forced_nbr is None else np.ascontiguousarray(
        forced_nbr.detach().cpu().numpy(), dtype=np.int32)
    lib().okv_propagate2_unit(_ptr(sv), _ptr(k), C.c_int32(n_prefix), C.c_int32(k.shape[1]), _ptr(s),
                              C.c_int32(topk_nodes), C.c_int32(m), C.c_int32(rounds),
                              C.c_double(decay), C.c_int32(signal), _ptr(fs), _ptr(fn), _ptr(src),
                              _ptr(nbr), _ptr(nbr_e))
    return (torch.from_numpy(s), torch.from_numpy(src[:topk_nodes]),
            torch.from_numpy(nbr[:topk_nodes]), torch.from_numpy(nbr_e[:topk_nodes]))


def propagate(K: torch.Tensor, scores: torch.Tensor, window: int, topk_nodes: int,
              neighbors: int, rounds: int, decay: float, signal: int = 0, reselect: int = 0):
    """All heads.  Returns (scores after T rounds fp32 [batch, Hkv, N], sources int32)."""
    sh = _shape(None, K, window)
    p = _params(sh, topk_nodes=topk_nodes, neighbors=neighbors, rounds=rounds, decay=decay,
                signal=signal, reselect=reselect)
    k = _f32(K)
    s = np.array(scores.detach().cpu().numpy(), dtype=np.float32, copy=True)
    src = np.zeros((sh.batch, sh.n_kv_heads, max(topk_nodes, 1)), dtype=np.int32)
    lib().okv_propagate(C.byref(p), _ptr(k), _ptr(s), _ptr(src) if topk_nodes > 0 else None)
    return torch.from_numpy(s), torch.from_numpy(src[..., :topk_nodes])


def select_gather(scores: torch.Tensor, K: torch.Tensor, V: torch.Tensor, window: int,
                  budget: int):
    """Top-B per head (ascending positions) and the compact cache [batch, Hkv, B+W, D]."""
    sh = _shape(None, K, window)
    p = _params(sh, budget=budget)
    s = np.ascontiguousarray(scores.detach().cpu().numpy(), dtype=np.float32)
    kr, eb = _raw(K)
    vr, _ = _raw(V)
    out_shape = (sh.batch, sh.n_kv_heads, budget + window, sh.head_dim)
    K_out = torch.empty(out_shape, dtype=K.dtype)
    V_out = torch.empty(out_shape, dtype=V.dtype)
    ko = K_out.view(torch.uint8).numpy().reshape(-1)
    vo = V_out.view(torch.uint8).numpy().reshape(-1)
    idx = np.empty((sh.batch, sh.n_kv_heads, budget), dtype=np.int32)
    lib().okv_select_gather(C.byref(p), _ptr(s), _ptr(kr), _ptr(vr), C.c_size_t(eb), _ptr(ko),
                            _ptr(vo), _ptr(idx))
    return K_out, V_out, torch.from_numpy(idx)


def compress(Qw: torch.Tensor, K: torch.Tensor, V: torch.Tensor, *, window: int, budget: int,
             pool_kernel: int, topk_nodes: int, neighbors: int, rounds: int, decay: float,
             pool_mode: int = 0, signal: int = 0, reselect: int = 0):
    """The whole path.  Returns (K_out, V_out, idx int32 [batch,Hkv,B], final scores fp32)."""
    sh = _shape(Qw, K, window)
    p = _params(sh, budget=budget, pool_kernel=pool_kernel, topk_nodes=topk_nodes,
                neighbors=neighbors, rounds=rounds, decay=decay, pool_mode=pool_mode,
                signal=signal, reselect=reselect)
    q, k = _f32(Qw), _f32(K)
    kr, eb = _raw(K)
    vr, _ = _raw(V)
    out_shape = (sh.batch, sh.n_kv_heads, budget + window, sh.head_dim)
    K_out = torch.empty(out_shape, dtype=K.dtype)
    V_out = torch.empty(out_shape, dtype=V.dtype)
    ko = K_out.view(torch.uint8).numpy().reshape(-1)
    vo = V_out.view(torch.uint8).numpy().reshape(-1)
    idx = np.empty((sh.batch, sh.n_kv_heads, budget), dtype=np.int32)
    s = np.empty((sh.batch, sh.n_kv_heads, sh.n_prefix), dtype=np.float32)
    lib().okv_compress(C.byref(p), _ptr(q), _ptr(k), _ptr(kr), _ptr(vr), C.c_size_t(eb),
                       _ptr(ko), _ptr(vo), _ptr(idx), _ptr(s))
    return K_out, V_out, torch.from_numpy(idx), torch.from_numpy(s)
