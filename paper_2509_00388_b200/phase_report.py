"""Per-kernel phase times of one compress step, from a library built with phase timing.

    python -m paper_2509_00388_b200.build --phases
    python -m paper_2509_00388_b200.phase_report [workload]

Loads libgraphkv_phases.so (its kernels stamp the global timer at the phase marks in their
sources), runs three warm-up and five timed calls of graphkv_compress on the named workload and
prints, per kernel, the mean and the largest time a CTA spent in each phase, in microseconds.
"""
from __future__ import annotations

import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
os.environ.setdefault("GRAPHKV_LIB", os.path.join(HERE, "libgraphkv_phases.so"))

import torch  # noqa: E402

from . import binding as gk  # noqa: E402
from . import workloads as wl  # noqa: E402

KERNELS = {0: "score_stats_tc", 1: "score_emit_tc", 2: "similarity_tc", 3: "pool_select_kernel",
           4: "finish_kernel (first CTA of a cluster)", 5: "score_fused_tc",
           6: "finish_kernel (other CTAs)"}


def main(name: str = "llama31_8b_32k", steps: int = 5) -> None:
    cfg = wl.CONFIGS[name]
    dev = torch.device("cuda:0")
    inp = {k: v.to(dev) for k, v in wl.make_inputs(cfg).items()}
    p = gk.make_params(inp["K"], Qw=inp["Qw"], V=inp["V"], window=cfg.window, budget=cfg.budget,
                       pool_kernel=cfg.pool_kernel, topk_nodes=cfg.topk_nodes,
                       neighbors=cfg.neighbors, rounds=cfg.rounds, decay=cfg.decay)
    ws = gk.alloc_workspace(p, dev)
    K_out, V_out, idx, _ = gk.alloc_outputs(p, inp["K"], want_scores=False)

    def call():
        gk.graphkv_compress(p, inp["Qw"], inp["K"], inp["V"], K_out, V_out, idx, None, ws)

    for _ in range(3):
        call()
    torch.cuda.synchronize()
    if gk.graphkv_phase_timing_read() is None:
        raise SystemExit("this library was built without phase timing: python -m paper_2509_00388_b200.build --phases")
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(steps):
        call()
    ev1.record()
    torch.cuda.synchronize()
    print(f"{name}: {1e3 * ev0.elapsed_time(ev1) / steps:.1f} us per step (instrumented build)")
    for k, (cnt, ph) in sorted(gk.graphkv_phase_timing_read().items()):
        print(f"{KERNELS.get(k, k)}: {cnt / steps:.0f} CTAs per step, whole CTA mean {ph[0][0] / 1e3:.2f} "
              f"max {ph[0][1] / 1e3:.2f} us")
        print("   mean:", " ".join(f"{m / 1e3:.2f}" for m, x in ph[1:] if x > 0))
        print("   max :", " ".join(f"{x / 1e3:.2f}" for m, x in ph[1:] if x > 0))


if __name__ == "__main__":
    main(*(sys.argv[1:2]))
