"""Seeded synthetic inputs for the GraphKV prefill-compression path.

This module only *draws inputs*: cluster-mixture keys with near-duplicates, window
queries aligned to a few clusters, values, and the per-layer budget ramp.  It holds
none of the method's arithmetic (no scores, similarities, selections) so that both
the CPU oracle's tests and the CUDA path's tests can share it without sharing any
of the computation under test.

The inputs stand in for prompts of a long-context benchmark pushed through
Llama-2-7B / Llama-3-8B / Mistral-7B (the paper's Experimental Setup): they take the
shapes (32 query heads, 8 KV heads, head_dim 128, 16K-128K tokens) and the qualitative
structure the paper's Observation section reports for real keys (high mean cosine
similarity inside groups of tokens, redundant high-importance tokens), not any item
of those suites.

Layout of every returned tensor (CPU, contiguous):
    Qw : [batch, n_q_heads,  W, D]   queries of the observation window
    K  : [batch, n_kv_heads, L, D]   keys,   L = N + W, rows [0,N) prefix, [N,L) window
    V  : [batch, n_kv_heads, L, D]   values, same layout
dtype bf16 (round-to-nearest-even from fp32) or fp32.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional, Sequence, Tuple

import numpy as np
import torch


@dataclass(frozen=True)
class GraphKVConfig:
    name: str
    batch: int              # independent sequences
    n_layers: int           # independent layers (each generated from its own seed)
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_prefix: int           # N: tokens that are candidates for eviction
    window: int             # W: observation-window queries / always-kept tokens
    budget: int             # B for layer 0 (see layer_budget for ramps)
    budget_last: Optional[int]  # if set: linear ramp budget -> budget_last over layers
    pool_kernel: int
    topk_nodes: int         # K_src
    neighbors: int          # m (0 = the library's adaptive rule)
    rounds: int             # T
    decay: float            # lambda
    dtype: str              # "bf16" | "f32"
    # generator constants
    n_clusters: int
    center_scale: float     # key = center_scale * c_z + noise_sigma * N(0, I)
    noise_sigma: float
    dup_frac: float         # share of prefix positions that copy an earlier key
    dup_sigma: float        # per-coordinate noise of such a copy
    q_clusters: int         # clusters each query head is aligned to
    q_scale: float          # query = q_scale * c_z + N(0, I)
    heavy_frac: float       # share of keys boosted along the mean query direction
    heavy_scale: float
    seed: int

    @property
    def seq_len(self) -> int:
        return self.n_prefix + self.window

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def layer_budget(self, layer: int) -> int:
        if self.budget_last is None or self.n_layers <= 1:
            return self.budget
        span = self.budget - self.budget_last
        return int(round(self.budget - span * layer / (self.n_layers - 1)))

    def torch_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32


_SQRT_D = float(np.sqrt(128.0))

CONFIGS: Dict[str, GraphKVConfig] = {}


def _register(cfg: GraphKVConfig) -> GraphKVConfig:
    CONFIGS[cfg.name] = cfg
    return cfg


# The five benchmark workloads.  Fields their definition leaves open
# (pool kernel where not given, decay everywhere, neighbours) take pool_kernel=7,
# decay=1.0 and the adaptive neighbour rule's value written out explicitly.
TINY = _register(GraphKVConfig(
    name="tiny", batch=1, n_layers=1, n_q_heads=1, n_kv_heads=1, head_dim=128,
    n_prefix=512, window=32, budget=64, budget_last=None, pool_kernel=7, topk_nodes=8,
    neighbors=4, rounds=1, decay=1.0, dtype="f32",
    n_clusters=16, center_scale=1.0, noise_sigma=0.1, dup_frac=0.20, dup_sigma=0.01,
    q_clusters=4, q_scale=6.0 * _SQRT_D, heavy_frac=0.0, heavy_scale=1.0, seed=0))

LLAMA_32K = _register(GraphKVConfig(
    name="llama31_8b_32k", batch=1, n_layers=1, n_q_heads=32, n_kv_heads=8, head_dim=128,
    n_prefix=32768, window=32, budget=512, budget_last=None, pool_kernel=7, topk_nodes=16,
    neighbors=32, rounds=2, decay=1.0, dtype="bf16",
    n_clusters=256, center_scale=2.0 * _SQRT_D, noise_sigma=1.0, dup_frac=0.10,
    dup_sigma=0.05, q_clusters=4, q_scale=6.0, heavy_frac=0.0, heavy_scale=1.0, seed=0))

MISTRAL_16K = _register(GraphKVConfig(
    name="mistral_7b_16k_32layers", batch=1, n_layers=32, n_q_heads=32, n_kv_heads=8,
    head_dim=128, n_prefix=16384, window=32, budget=2048, budget_last=None, pool_kernel=7,
    topk_nodes=16, neighbors=16, rounds=3, decay=1.0, dtype="bf16",
    n_clusters=256, center_scale=2.0 * _SQRT_D, noise_sigma=1.0, dup_frac=0.10,
    dup_sigma=0.05, q_clusters=4, q_scale=6.0, heavy_frac=0.01, heavy_scale=4.0, seed=0))

PYRAMID_32K = _register(GraphKVConfig(
    name="pyramidkv_32k_32layers", batch=1, n_layers=32, n_q_heads=32, n_kv_heads=8,
    head_dim=128, n_prefix=32768, window=32, budget=2048, budget_last=128, pool_kernel=7,
    topk_nodes=16, neighbors=32, rounds=2, decay=1.0, dtype="bf16",
    n_clusters=256, center_scale=2.0 * _SQRT_D, noise_sigma=1.0, dup_frac=0.10,
    dup_sigma=0.05, q_clusters=4, q_scale=6.0, heavy_frac=0.0, heavy_scale=1.0, seed=0))

LONG_128K = _register(GraphKVConfig(
    name="long_128k_batch4", batch=4, n_layers=1, n_q_heads=32, n_kv_heads=8, head_dim=128,
    n_prefix=131072, window=64, budget=4096, budget_last=None, pool_kernel=7, topk_nodes=32,
    neighbors=32, rounds=4, decay=1.0, dtype="bf16",
    n_clusters=256, center_scale=2.0 * _SQRT_D, noise_sigma=1.0, dup_frac=0.30,
    dup_sigma=0.05, q_clusters=4, q_scale=6.0, heavy_frac=0.0, heavy_scale=1.0, seed=0))

CONFIG_ORDER: Tuple[str, ...] = (
    "tiny", "llama31_8b_32k", "mistral_7b_16k_32layers", "pyramidkv_32k_32layers",
    "long_128k_batch4")


def scaled(cfg: GraphKVConfig, **changes) -> GraphKVConfig:
    """A copy of cfg with some fields replaced (smaller N for parity tests, etc.)."""
    return replace(cfg, **changes)


def _unit_rows(rng: np.random.Generator, n: int, d: int) -> np.ndarray:
    c = rng.standard_normal((n, d), dtype=np.float32)
    c /= np.linalg.norm(c, axis=1, keepdims=True)
    return c


def _mixture_rows(rng: np.random.Generator, centers: np.ndarray, n_rows: int, n_prefix: int,
                  cfg: GraphKVConfig) -> np.ndarray:
    """n_rows cluster-mixture vectors; the first n_prefix rows get near-duplicates."""
    d = centers.shape[1]
    z = rng.integers(0, centers.shape[0], size=n_rows)
    x = rng.standard_normal((n_rows, d), dtype=np.float32)
    x *= np.float32(cfg.noise_sigma)
    x += np.float32(cfg.center_scale) * centers[z]
    n_dup = int(round(cfg.dup_frac * n_prefix))
    if n_dup > 0 and n_prefix > 1:
        # Position 0 is never a copy; a copy takes an earlier *original* position as model.
        dup_pos = np.sort(rng.choice(np.arange(1, n_prefix), size=min(n_dup, n_prefix - 1),
                                     replace=False))
        is_dup = np.zeros(n_prefix, dtype=bool)
        is_dup[dup_pos] = True
        orig_pos = np.flatnonzero(~is_dup)
        n_before = np.searchsorted(orig_pos, dup_pos, side="left")  # originals earlier than p
        pick = (rng.random(dup_pos.shape[0]) * n_before).astype(np.int64)
        src = orig_pos[np.minimum(pick, n_before - 1)]
        jitter = rng.standard_normal((dup_pos.shape[0], d), dtype=np.float32)
        x[dup_pos] = x[src] + np.float32(cfg.dup_sigma) * jitter
    return x


def _to_tensor(x: np.ndarray, cfg: GraphKVConfig) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32))
    return t.to(cfg.torch_dtype()).contiguous()


def make_inputs(cfg: GraphKVConfig, layer: int = 0,
                sequences: Optional[Sequence[int]] = None) -> Dict[str, torch.Tensor]:
    """Draw Qw, K, V for one layer.  Seed of a (layer, sequence) unit is
    cfg.seed + 1000*layer + sequence, so units can be generated independently."""
    seqs = list(range(cfg.batch)) if sequences is None else list(sequences)
    d, n, w, ell = cfg.head_dim, cfg.n_prefix, cfg.window, cfg.seq_len
    g = cfg.group
    q_all = np.empty((len(seqs), cfg.n_q_heads, w, d), dtype=np.float32)
    k_all = np.empty((len(seqs), cfg.n_kv_heads, ell, d), dtype=np.float32)
    v_all = np.empty((len(seqs), cfg.n_kv_heads, ell, d), dtype=np.float32)
    for bi, seq in enumerate(seqs):
        rng = np.random.default_rng(np.random.PCG64(cfg.seed + 1000 * layer + seq))
        for h in range(cfg.n_kv_heads):
            centers = _unit_rows(rng, cfg.n_clusters, d)
            k = _mixture_rows(rng, centers, ell, n, cfg)
            # queries of the G heads that share this KV head
            for gi in range(g):
                zq = rng.choice(cfg.n_clusters, size=min(cfg.q_clusters, cfg.n_clusters),
                                replace=False)
                pick = zq[rng.integers(0, zq.shape[0], size=w)]
                q = rng.standard_normal((w, d), dtype=np.float32)
                q += np.float32(cfg.q_scale) * centers[pick]
                q_all[bi, h * g + gi] = q
            if cfg.heavy_frac > 0.0:
                # heavy hitters: boost the component along the head's mean query direction
                u = q_all[bi, h * g:(h + 1) * g].reshape(-1, d).mean(axis=0)
                u /= max(float(np.linalg.norm(u)), 1e-12)
                n_heavy = max(1, int(round(cfg.heavy_frac * n)))
                pos = rng.choice(n, size=n_heavy, replace=False)
                comp = k[pos] @ u
                k[pos] += np.float32(cfg.heavy_scale - 1.0) * comp[:, None] * u[None, :]
            k_all[bi, h] = k
            v_centers = _unit_rows(rng, cfg.n_clusters, d)
            v_all[bi, h] = _mixture_rows(rng, v_centers, ell, n, cfg)
    return {"Qw": _to_tensor(q_all, cfg), "K": _to_tensor(k_all, cfg),
            "V": _to_tensor(v_all, cfg)}


def make_scores(n_rows: int, n: int, seed: int, tie_frac: float = 0.0) -> torch.Tensor:
    """Non-negative fp32 score rows with a heavy tail (for testing selection stages alone).
    tie_frac > 0 plants exact repeats of earlier values to exercise tie-breaking."""
    rng = np.random.default_rng(np.random.PCG64(seed))
    s = np.exp(3.0 * rng.standard_normal((n_rows, n))).astype(np.float32)
    n_tie = int(round(tie_frac * n))
    if n_tie > 0 and n > 1:
        for r in range(n_rows):
            dst = rng.choice(n, size=n_tie, replace=False)
            src = rng.integers(0, n, size=n_tie)
            s[r, dst] = s[r, src]
    return torch.from_numpy(s)
