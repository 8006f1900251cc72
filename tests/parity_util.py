"""Comparison procedures shared by the GPU parity tests and the smoke check.

Tolerances: scores within 2e-3 relative (the fp32 tensor-core path measures about twenty times
inside it); retained index sets bit-exact wherever the selection-boundary margin exceeds that
tolerance, swaps inside the near-tie band counted, overall overlap >= 99.9 %; gathered K/V
bit-exact.

Because every selection is a discrete decision, stages are compared with teacher forcing:
  * sources: the oracle's top-k on the GPU's own fp32 scores must equal the GPU's sources exactly;
  * neighbourhoods (Eq. 3): the GPU's lists are read back and each must be a valid top-m of the
    oracle's fp64 cosines -- equal to the oracle's own pick except for members whose cosine lies
    within fp32 resolution (EDGE_TIE) of the m-th largest; the cosines the GPU reports must match;
  * decay (Eq. 5): the oracle is restarted from the GPU's scores, sources and neighbour lists and
    every element of every head must then agree within the score tolerance.
"""
from __future__ import annotations

import json
import os
from dataclasses import dataclass, field
from typing import Dict, List

import numpy as np
import torch

from oracle import graphkv_oracle as okv

SCORE_RTOL = 2e-3          # stated tolerance on scores
SCORE_FLOOR = 1e-6         # floor of the denominator, relative to the head's largest score
EDGE_TIE = 4e-6            # cosine margin below which fp32 cannot be expected to rank alike
MIN_OVERLAP = 0.999
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@dataclass
class Report:
    max_score_rel_err: float = 0.0
    max_final_rel_err: float = 0.0
    max_edge_abs_err: float = 0.0
    near_tie_swaps: int = 0
    neighbour_near_tie_swaps: int = 0
    neighbour_tie_heads: int = 0
    source_near_tie_heads: int = 0
    heads: int = 0
    kept_total: int = 0
    kept_common: int = 0
    notes: List[str] = field(default_factory=list)

    @property
    def overlap(self) -> float:
        return self.kept_common / max(self.kept_total, 1)

    def as_dict(self) -> Dict[str, float]:
        return {"heads": self.heads,
                "max_score_rel_err": self.max_score_rel_err,
                "max_final_rel_err": self.max_final_rel_err,
                "max_edge_abs_err": self.max_edge_abs_err,
                "near_tie_swaps": self.near_tie_swaps,
                "neighbour_near_tie_swaps": self.neighbour_near_tie_swaps,
                "neighbour_tie_heads": self.neighbour_tie_heads,
                "source_near_tie_heads": self.source_near_tie_heads,
                "set_overlap": self.overlap,
                "notes": self.notes[:32]}

    def write(self, name: str) -> None:
        """Leaves the counters on file: parity_<name>.json in the repository's scratch output folder."""
        out = os.path.join(ROOT, "gpurun_out")
        try:
            os.makedirs(out, exist_ok=True)
            with open(os.path.join(out, f"parity_{name}.json"), "w") as f:
                json.dump(self.as_dict(), f, indent=1)
        except OSError:
            pass


def score_rel_err(got: torch.Tensor, want: torch.Tensor) -> float:
    """max |g - o| / max(|o|, floor) with floor = 1e-6 * max_j o_j, per head (last dim)."""
    g = got.double().reshape(-1, got.shape[-1]).numpy()
    o = want.double().reshape(-1, want.shape[-1]).numpy()
    floor = SCORE_FLOOR * np.abs(o).max(axis=1, keepdims=True)
    return float((np.abs(g - o) / np.maximum(np.abs(o), floor)).max())


def check_neighbourhoods(Kh: torch.Tensor, n: int, m: int, src: np.ndarray, nbr: np.ndarray,
                         nbr_e: np.ndarray, rep: Report, where: str) -> bool:
    """Eq. 3 on one head: every GPU list is a valid top-m of the oracle's cosines of its source.
    Returns True when some list differs from the oracle's own pick (inside the margin)."""
    differs = False
    for a, i in enumerate(src.tolist()):
        e = okv.edges_unit(Kh, n, i).numpy()
        got = nbr[a]
        assert got.min() >= 0 and got.max() < n and i not in got, f"{where} src {i}: bad neighbour"
        assert len(set(got.tolist())) == m, f"{where} src {i}: repeated neighbour"
        err = float(np.abs(nbr_e[a].astype(np.float64) - e[got]).max())
        rep.max_edge_abs_err = max(rep.max_edge_abs_err, err)
        assert err <= EDGE_TIE, f"{where} src {i}: reported cosine off by {err}"
        want = okv.topk(torch.from_numpy(e.astype(np.float32)), m, skip=i).numpy()
        diff = set(got.tolist()) ^ set(want.tolist())
        if diff:
            boundary = float(e[want].min())            # the oracle's m-th largest cosine
            worst = max(abs(float(e[j]) - boundary) for j in diff)
            assert worst <= EDGE_TIE, \
                f"{where} src {i}: neighbour sets differ outside the margin ({worst:.2e})"
            rep.neighbour_near_tie_swaps += len(diff) // 2
            differs = True
    return differs


def check_compress(gpu: Dict[str, torch.Tensor], Qw: torch.Tensor, K: torch.Tensor,
                   V: torch.Tensor, *, window: int, budget: int, pool_kernel: int,
                   topk_nodes: int, neighbors: int, rounds: int, decay: float,
                   strict_overlap: bool = True) -> Report:
    """gpu: CPU copies of the GPU path's stage outputs for the same inputs:
         scores0 [b,h,N]  after graphkv_score
         src     [b,h,K_src] from graphkv_propagate (may be absent if K_src == 0)
         nbr, nbr_e [b,h,K_src,m] from graphkv_read_neighbors (when a graph was built)
         scores  [b,h,N]  after graphkv_propagate
         idx     [b,h,B], K_out, V_out from graphkv_select_gather
    Raises AssertionError on a parity violation; returns the counters otherwise."""
    rep = Report()
    b, hkv, ell, d = K.shape
    n = ell - window
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
            rep.heads += 1
            where = f"b={bi} h={h}"
            s0 = gpu["scores0"][bi, h]
            nbr_differs = False
            # (b) Eq. 2 restarted from the GPU's scores: identical fp32 values, identical pick
            if topk_nodes > 0:
                want_src = okv.topk(s0, topk_nodes).numpy()
                got_src = gpu["src"][bi, h].numpy()
                assert sorted(got_src.tolist()) == sorted(want_src.tolist()), \
                    f"sources differ on identical fp32 scores ({where})"
            if propagating:
                # (c) Eq. 3: the GPU's neighbour lists, then Eq. 5 forced onto them
                g_src = gpu["src"][bi, h].numpy()
                g_nbr = gpu["nbr"][bi, h].numpy()
                nbr_differs = check_neighbourhoods(K[bi, h], n, m, g_src, g_nbr,
                                                   gpu["nbr_e"][bi, h].numpy(), rep, where)
                if nbr_differs:
                    rep.neighbour_tie_heads += 1
                    rep.notes.append(f"{where}: neighbour near-tie")
                o_s, _, _, _ = okv.propagate_unit(
                    K[bi, h], s0, n, topk_nodes, neighbors, rounds, decay,
                    forced_src=gpu["src"][bi, h], forced_nbr=gpu["nbr"][bi, h])
                err = score_rel_err(gpu["scores"][bi, h][None], o_s[None])
                rep.max_final_rel_err = max(rep.max_final_rel_err, err)
                assert err <= SCORE_RTOL, f"propagated score rel err {err} ({where})"
                assert torch.all(gpu["scores"][bi, h] <= s0), "a score increased under decay"
                changed = set(torch.nonzero(gpu["scores"][bi, h] != s0).flatten().tolist())
                assert changed <= set(g_nbr.reshape(-1).tolist()), \
                    f"a score outside every neighbourhood changed ({where})"
            else:
                assert torch.equal(gpu["scores"][bi, h], s0), "scores changed without propagation"

            # (d) step (IV) on the GPU's final scores: bit-exact
            want_idx = np.sort(okv.topk(gpu["scores"][bi, h], budget).numpy())
            got_idx = gpu["idx"][bi, h].numpy()
            assert np.array_equal(got_idx, want_idx), f"selection differs ({where})"
            assert len(set(got_idx.tolist())) == budget and got_idx.min() >= 0 and got_idx.max() < n

            # (e) gather: bit-exact, window retained
            ii = torch.from_numpy(got_idx).long()
            for name, X in (("K_out", K), ("V_out", V)):
                want = torch.cat([X[bi, h, ii], X[bi, h, n:]])
                assert torch.equal(gpu[name][bi, h].view(torch.uint8).reshape(-1),
                                   want.contiguous().view(torch.uint8).reshape(-1)), \
                    f"{name} not bit-exact ({where})"

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
                if outside and not nbr_differs:
                    # only a flip at the source boundary can explain it, and only sources whose
                    # oracle scores sit within the tolerance of the K_src-th score can flip
                    o_s0 = o_scores0[bi, h].double().numpy()
                    o_src_free = set(okv.topk(o_scores0[bi, h], topk_nodes).tolist()) \
                        if topk_nodes > 0 else set()
                    g_src = set(gpu["src"][bi, h].tolist()) if topk_nodes > 0 else set()
                    flipped = o_src_free ^ g_src
                    assert flipped, \
                        f"kept sets differ outside the near-tie band ({where}): {outside[:8]}"
                    kth = np.sort(o_s0)[::-1][topk_nodes - 1]
                    tol = SCORE_RTOL * max(abs(kth), SCORE_FLOOR * o_s0.max())
                    far = [j for j in flipped if abs(o_s0[j] - kth) > tol]
                    assert not far, f"sources {far[:8]} flipped outside the tolerance ({where})"
                    rep.source_near_tie_heads += 1
                    rep.notes.append(f"{where}: source near-tie")
    if strict_overlap:
        assert rep.overlap >= MIN_OVERLAP, f"set overlap {rep.overlap}"
    return rep
