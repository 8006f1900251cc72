"""Comparison procedures shared by the GPU parity tests and the smoke check.

Tolerances: scores within 2e-3 relative (the fp32 tensor-core path is three orders inside it); retained index
sets bit-exact wherever the selection-boundary margin exceeds that tolerance, swaps inside the
near-tie band counted, overall overlap >= 99.9 %; gathered K/V bit-exact.

Because every selection is a discrete decision, stages are compared with teacher forcing: the
oracle is restarted from the GPU's own fp32 stage outputs, on which its fp32 ranking decisions
must coincide with the GPU's exactly; only where the oracle's own neighbour margin is below
fp32 resolution is a head reported as an "upstream near-tie" instead of compared strictly.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List

import numpy as np
import torch

from oracle import graphkv_oracle as okv

SCORE_RTOL = 2e-3          # stated tolerance on scores
SCORE_FLOOR = 1e-6         # floor of the denominator, relative to the head's largest score
EDGE_TIE = 4e-6            # cosine margin below which fp32 cannot be expected to rank alike
MIN_OVERLAP = 0.999


@dataclass
class Report:
    max_score_rel_err: float = 0.0
    max_final_rel_err: float = 0.0
    near_tie_swaps: int = 0
    upstream_near_tie_heads: int = 0
    kept_total: int = 0
    kept_common: int = 0
    notes: List[str] = field(default_factory=list)

    @property
    def overlap(self) -> float:
        return self.kept_common / max(self.kept_total, 1)

    def as_dict(self) -> Dict[str, float]:
        return {"max_score_rel_err": self.max_score_rel_err,
                "max_final_rel_err": self.max_final_rel_err,
                "near_tie_swaps": self.near_tie_swaps,
                "upstream_near_tie_heads": self.upstream_near_tie_heads,
                "set_overlap": self.overlap}


def score_rel_err(got: torch.Tensor, want: torch.Tensor) -> float:
    """max |g - o| / max(|o|, floor) with floor = 1e-6 * max_j o_j, per head (last dim)."""
    g = got.double().reshape(-1, got.shape[-1]).numpy()
    o = want.double().reshape(-1, want.shape[-1]).numpy()
    floor = SCORE_FLOOR * np.abs(o).max(axis=1, keepdims=True)
    return float((np.abs(g - o) / np.maximum(np.abs(o), floor)).max())


def neighbour_margin(nbr_e_sorted_desc: np.ndarray, runner_up: float) -> float:
    return float(nbr_e_sorted_desc[-1] - runner_up)


def check_compress(gpu: Dict[str, torch.Tensor], Qw: torch.Tensor, K: torch.Tensor,
                   V: torch.Tensor, *, window: int, budget: int, pool_kernel: int,
                   topk_nodes: int, neighbors: int, rounds: int, decay: float,
                   strict_overlap: bool = True) -> Report:
    """gpu: CPU copies of the GPU path's stage outputs for the same inputs:
         scores0 [b,h,N]  after graphkv_score
         src     [b,h,K_src] from graphkv_propagate (may be absent if K_src == 0)
         scores  [b,h,N]  after graphkv_propagate
         idx     [b,h,B], K_out, V_out from graphkv_select_gather
    Raises AssertionError on a parity violation; returns the counters otherwise."""
    rep = Report()
    b, hkv, ell, d = K.shape
    n = ell - window
    g = Qw.shape[1] // hkv
    m = okv.resolve_neighbors(n, neighbors)

    # (a) step (I): scores against the oracle
    o_scores0 = okv.score(Qw, K, window, pool_kernel)
    rep.max_score_rel_err = score_rel_err(gpu["scores0"], o_scores0)
    assert rep.max_score_rel_err <= SCORE_RTOL, f"score rel err {rep.max_score_rel_err}"

    # pure-oracle end-to-end result for the set-overlap statement
    _, _, o_idx, o_final = okv.compress(Qw, K, V, window=window, budget=budget,
                                        pool_kernel=pool_kernel, topk_nodes=topk_nodes,
                                        neighbors=neighbors, rounds=rounds, decay=decay)

    propagating = topk_nodes > 0 and rounds > 0 and m > 0
    for bi in range(b):
        for h in range(hkv):
            s0 = gpu["scores0"][bi, h]
            upstream_tie = False
            # (b)+(c) steps (II)+(III), restarted from the GPU's scores
            if topk_nodes > 0:
                want_src = okv.topk(s0, topk_nodes).numpy()
                got_src = gpu["src"][bi, h].numpy()
                assert sorted(got_src.tolist()) == sorted(want_src.tolist()), \
                    f"sources differ on identical fp32 scores (b={bi}, h={h})"
            if propagating:
                o_s, o_src, o_nbr, o_nbr_e = okv.propagate_unit(
                    K[bi, h], s0, n, topk_nodes, neighbors, rounds, decay)
                # is any neighbourhood boundary within fp32 resolution?
                if m < n - 1:
                    for a, i in enumerate(o_src.tolist()):
                        e = okv.edges_unit(K[bi, h], n, i).numpy()
                        e[i] = -np.inf
                        e[o_nbr[a].numpy()] = -np.inf
                        if o_nbr_e[a].numpy().min() - e.max() < EDGE_TIE:
                            upstream_tie = True
                            break
                err = score_rel_err(gpu["scores"][bi, h][None], o_s[None])
                if upstream_tie:
                    rep.upstream_near_tie_heads += 1
                    rep.notes.append(f"b={bi} h={h}: neighbour near-tie, final rel err {err:.2e}")
                else:
                    rep.max_final_rel_err = max(rep.max_final_rel_err, err)
                    assert err <= SCORE_RTOL, f"propagated score rel err {err} (b={bi}, h={h})"
                assert torch.all(gpu["scores"][bi, h] <= s0), "a score increased under decay"
                changed = int((gpu["scores"][bi, h] != s0).sum())
                assert changed <= topk_nodes * m, f"{changed} scores changed > K_src*m"
            else:
                assert torch.equal(gpu["scores"][bi, h], s0), "scores changed without propagation"

            # (d) step (IV) on the GPU's final scores: bit-exact
            want_idx = np.sort(okv.topk(gpu["scores"][bi, h], budget).numpy())
            got_idx = gpu["idx"][bi, h].numpy()
            assert np.array_equal(got_idx, want_idx), f"selection differs (b={bi}, h={h})"
            assert len(set(got_idx.tolist())) == budget and got_idx.min() >= 0 and got_idx.max() < n

            # (e) gather: bit-exact, window retained
            ii = torch.from_numpy(got_idx).long()
            for name, X in (("K_out", K), ("V_out", V)):
                want = torch.cat([X[bi, h, ii], X[bi, h, n:]])
                assert torch.equal(gpu[name][bi, h].view(torch.uint8).reshape(-1),
                                   want.contiguous().view(torch.uint8).reshape(-1)), \
                    f"{name} not bit-exact (b={bi}, h={h})"

            # (f) free-running comparison with the oracle's own end-to-end result
            oi = set(o_idx[bi, h].tolist())
            gi = set(got_idx.tolist())
            rep.kept_total += budget
            rep.kept_common += len(oi & gi)
            diff = oi ^ gi
            if diff:
                of = o_final[bi, h].double().numpy()
                boundary = np.sort(of)[::-1][budget - 1]
                band = SCORE_RTOL * max(abs(boundary), SCORE_FLOOR * of.max())
                outside = [j for j in diff if abs(of[j] - boundary) > band]
                rep.near_tie_swaps += len(diff) // 2
                if outside and not upstream_tie:
                    # a source flip upstream also explains it: compare the source sets
                    o_src_free = set(okv.topk(o_scores0[bi, h], topk_nodes).tolist()) \
                        if topk_nodes > 0 else set()
                    g_src = set(gpu["src"][bi, h].tolist()) if topk_nodes > 0 else set()
                    if o_src_free != g_src:
                        rep.upstream_near_tie_heads += 1
                        rep.notes.append(f"b={bi} h={h}: source near-tie")
                    else:
                        raise AssertionError(
                            f"kept sets differ outside the near-tie band (b={bi}, h={h}): {outside[:8]}")
    if strict_overlap:
        assert rep.overlap >= MIN_OVERLAP, f"set overlap {rep.overlap}"
    return rep
