#!/usr/bin/env python
"""Benchmark of the GraphKV prefill-compression path on B200.

One step = one call of `graphkv_compress` (scores -> graph -> decay rounds -> top-B -> gather)
on one layer of the Llama-3.1-8B-shaped workload (32 query / 8 KV heads, head_dim 128,
N = 32768 prefix tokens, window 32, budget 512, 16 source nodes, 2 rounds), bf16, synthetic
seeded inputs.  Metric: context tokens per second per layer, all heads (batch * N / step time).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Under torchrun (N > 1) every rank runs an independent replica on its own GPU (the path has no
exchange step); the timed region is bracketed by a barrier and a device synchronise, the step
time is the maximum over ranks and the value is the sum of all ranks' tokens over that time.
`--impl reference` times the CPU oracle on the host cores instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time
from collections import defaultdict

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2509_00388_b200 import workloads as wl  # noqa: E402

METRIC = "prefill KV-compress context tokens/sec per layer (all heads)"
UNIT = "tokens/s"
ROTATING_SETS = 4          # distinct device copies of the inputs; 4 x 67 MB of K > 126 MB L2
FALLBACK_HBM_GBS = 6650.0


def cfg_kwargs(cfg, layer=0):
    return dict(window=cfg.window, budget=cfg.layer_budget(layer), pool_kernel=cfg.pool_kernel,
                topk_nodes=cfg.topk_nodes, neighbors=cfg.neighbors, rounds=cfg.rounds,
                decay=cfg.decay)


def config_dict(cfg, extra=None):
    d = {"workload": cfg.name, "batch": cfg.batch, "n_q_heads": cfg.n_q_heads,
         "n_kv_heads": cfg.n_kv_heads, "head_dim": cfg.head_dim, "n_prefix": cfg.n_prefix,
         "window": cfg.window, "budget": cfg.budget, "pool_kernel": cfg.pool_kernel,
         "topk_nodes": cfg.topk_nodes, "neighbors": cfg.neighbors, "rounds": cfg.rounds,
         "decay": cfg.decay, "parallelism": "replicas"}
    if extra:
        d.update(extra)
    return d


# ---- algorithmic bytes -------------------------------------------------------------------------
def algorithmic_bytes(cfg, kernel: str) -> float:
    """Bytes a kernel must move per launch for one layer of cfg (inputs it has to read once and
    outputs it has to write once; on-chip intermediates are not counted)."""
    e = 2 if cfg.dtype == "bf16" else 4
    units = cfg.batch * cfg.n_kv_heads
    N, L, D, W = cfg.n_prefix, cfg.seq_len, cfg.head_dim, cfg.window
    B, Ks = cfg.budget, cfg.topk_nodes
    m = cfg.neighbors
    k_sweep = units * L * D * e
    q_bytes = cfg.batch * cfg.n_q_heads * W * D * e
    row = 4 * units * N
    table = {
        "score_stats": k_sweep + q_bytes,
        "score_emit": units * N * D * e + q_bytes + row,
        "score_fused": k_sweep + q_bytes + row,
        "pool_max": 2 * row,
        "pool_select_sources": 2 * row + 4 * units * Ks,
        "decay_select_gather": 2 * row + 4 * units * B + 4 * units * (B + W) * D * e,
        "select_gather": row + 4 * units * B + 4 * units * (B + W) * D * e,
        "select_sources": row + 4 * units * Ks,
        "similarity": units * N * D * e + units * Ks * D * e,
        "select_neighbors": 0.0,
        "decay_rounds": 8 * units * Ks * m * 3,
        "select_budget": row + 4 * units * B,
        "gather_rows": 4 * units * (B + W) * D * e,
    }
    for key, val in table.items():
        if kernel.startswith(key):
            return float(val)
    return 0.0


# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu capture
# summarised in profiles/kernels_llama31_8b_32k_ncu_full.md; cold cache.  Only for the workload
# and kernels that capture covers; anything else reports null.
NCU_TRAFFIC = {"llama31_8b_32k": {"score_stats_tc": 67.86e6, "score_emit_tc": 67.87e6,
                                  "pool_select_sources": 1.18e6, "similarity_tc": 67.66e6,
                                  "decay_select_gather": 4.66e6}}


def path_bytes(cfg) -> float:
    """Algorithmic bytes of the whole path per layer: two sweeps of K (sources depend on all
    scores), the window queries, three passes over the fp32 score rows, the K/V gather."""
    e = 2 if cfg.dtype == "bf16" else 4
    units = cfg.batch * cfg.n_kv_heads
    return float(2 * units * cfg.seq_len * cfg.head_dim * e
                 + cfg.batch * cfg.n_q_heads * cfg.window * cfg.head_dim * e
                 + 12 * units * cfg.n_prefix
                 + 4 * units * (cfg.budget + cfg.window) * cfg.head_dim * e)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ---- clocks ------------------------------------------------------------------------------------
class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read-only) while the GPU works."""

    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap",
               0x8: "hw_slowdown", 0x10: "sync_boost", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
               0x100: "display_clock_setting"}

    def __init__(self, index: int, period_s: float = 0.001):
        self.samples, self.mask, self.max_mhz = [], 0, None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None
        self.period = period_s

    def _run(self):
        while not self._stop.is_set():
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
                self.mask |= int(self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        s = sorted(self.samples)
        reasons = [name for bit, name in self.REASONS.items()
                   if self.mask & bit and name != "gpu_idle"]
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(s)}


def visible_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ---- distributed plumbing ------------------------------------------------------------------------
def dist_setup(n_gpus: int):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        if not dist.is_initialized():
            backend = "nccl" if torch.cuda.is_available() else "gloo"
            dist.init_process_group(backend=backend)
    return world, rank, local


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(x: float, world: int, device) -> float:
    if world <= 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# ---- the oracle arm ------------------------------------------------------------------------------
def time_oracle(cfg, inp, repeats: int):
    from oracle import graphkv_oracle as okv
    kw = cfg_kwargs(cfg)
    okv.compress(inp["Qw"][:1, :cfg.group], inp["K"][:1, :1, :cfg.window + 64],
                 inp["V"][:1, :1, :cfg.window + 64], window=cfg.window, budget=8, pool_kernel=1,
                 topk_nodes=0, neighbors=0, rounds=0, decay=1.0)      # load the library
    times = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        okv.compress(inp["Qw"], inp["K"], inp["V"], **kw)
        times.append(time.perf_counter() - t0)
    return times, okv.num_threads()


def run_reference(args, cfg):
    # rank 0 alone works; no process group is needed for that
    if int(os.environ.get("RANK", "0")) != 0:
        return
    inp = wl.make_inputs(cfg)
    steps = max(1, min(args.steps, 20))
    warm = max(0, min(args.warmup, 2))
    time_oracle(cfg, inp, warm) if warm else None
    times, cores = time_oracle(cfg, inp, steps)
    mean = sum(times) / len(times)
    value = cfg.batch * cfg.n_prefix / mean
    sample = f"one full layer of {cfg.name} per step (all {cfg.n_kv_heads} KV heads)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
            "n_gpus": args.gpus, "steps": steps, "warmup": warm, "ms_per_step": mean * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": config_dict(cfg),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ---- our arm -----------------------------------------------------------------------------------
def run_ours(args, cfg):
    world, rank, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the CUDA path has no CPU fallback)")
    from paper_2509_00388_b200 import binding as gk
    gk.lib()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    kw = cfg_kwargs(cfg)

    inp = wl.make_inputs(cfg)
    host = {k: v.pin_memory() for k, v in inp.items()}
    sets = []
    for _ in range(ROTATING_SETS):
        sets.append({k: v.to(dev, non_blocking=True).clone() for k, v in host.items()})
    p = gk.make_params(sets[0]["K"], Qw=sets[0]["Qw"], V=sets[0]["V"], **kw)
    ws = gk.alloc_workspace(p, dev)
    K_out, V_out, idx, _ = gk.alloc_outputs(p, sets[0]["K"], want_scores=False)
    torch.cuda.synchronize(dev)

    def step(i):
        s = sets[i % ROTATING_SETS]
        gk.graphkv_compress(p, s["Qw"], s["K"], s["V"], K_out, V_out, idx, None, ws)

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize(dev)
    assert gk.graphkv_read_status(ws) == gk.OK

    # ---- timed region: K steps, inputs resident in HBM ----
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = gk.graphkv_launch_count()
    barrier(world)
    torch.cuda.synchronize(dev)
    with ClockSampler(visible_gpu_index(local)) as clocks:
        ev0.record()
        for i in range(args.steps):
            step(i)
        ev1.record()
        torch.cuda.synchronize(dev)
    barrier(world)
    launches = gk.graphkv_launch_count() - launches0
    ms_total = max_over_ranks(ev0.elapsed_time(ev1), world, dev)
    ms_step = ms_total / args.steps
    tokens_per_step = cfg.batch * cfg.n_prefix
    value = world * tokens_per_step / (ms_step * 1e-3)

    # ---- per-kernel durations: the same K steps again with event pairs around every launch ----
    gk.graphkv_trace_enable(True)
    for i in range(args.steps):
        step(i)
    torch.cuda.synchronize(dev)
    gk.graphkv_trace_enable(False)
    per_kernel = defaultdict(list)
    for name, ms in gk.graphkv_trace_read(args.steps * 32 + 64):
        per_kernel[name].append(ms)
    kernels = {n: {"launches_per_step": len(v) / args.steps, "avg_ms": sum(v) / len(v),
                   "ms_per_step": sum(v) / args.steps} for n, v in per_kernel.items()}
    top = max(kernels, key=lambda n: kernels[n]["ms_per_step"])
    peak, peak_kind = measured_peak()
    top_bytes = algorithmic_bytes(cfg, top)
    achieved = top_bytes / (kernels[top]["avg_ms"] * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": top, "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak,
                "traffic": NCU_TRAFFIC.get(cfg.name, {}).get(top),
                "peak_source": f"{peak_kind} copy bandwidth",
                "algorithmic_bytes_per_launch": top_bytes,
                "avg_launch_ms": kernels[top]["avg_ms"],
                "timing": "CUDA event pairs around every launch, second pass of the same steps",
                "whole_path": {"algorithmic_bytes_per_step": path_bytes(cfg),
                               "achieved_gbs": path_bytes(cfg) / (ms_step * 1e-3) / 1e9,
                               "frac_of_peak": path_bytes(cfg) / (ms_step * 1e-3) / 1e9 / peak,
                               "frac_of_8tbs": path_bytes(cfg) / (ms_step * 1e-3) / 1e9 / 8000.0},
                "kernels": {n: round(k["ms_per_step"], 5) for n, k in kernels.items()},
                "per_kernel": {n: {"algorithmic_bytes": algorithmic_bytes(cfg, n),
                                   "achieved_gbs": round(algorithmic_bytes(cfg, n) / (k["avg_ms"] * 1e-3) / 1e9, 1),
                                   "frac": round(algorithmic_bytes(cfg, n) / (k["avg_ms"] * 1e-3) / 1e9 / peak, 4)}
                               for n, k in kernels.items()}}

    # ---- end to end: host buffers in, compact cache out, copies inside the timed region ----
    e2e_steps = max(3, min(args.steps, 50))
    hK = torch.empty(K_out.shape, dtype=K_out.dtype).pin_memory()
    hV = torch.empty(V_out.shape, dtype=V_out.dtype).pin_memory()
    hI = torch.empty(idx.shape, dtype=idx.dtype).pin_memory()
    dst = sets[0]

    # Qw and K are copied to the device (the sweeps read K three times); V stays in pinned host
    # memory and the gather reads its B+W kept rows per head through the mapping; the compact
    # cache and the indices are written to pinned host memory by the gather itself.
    def e2e_step():
        for k in ("Qw", "K"):
            dst[k].copy_(host[k], non_blocking=True)
        gk.graphkv_compress(p, dst["Qw"], dst["K"], host["V"], hK, hV, hI, None, ws)

    for _ in range(2):
        e2e_step()
    torch.cuda.synchronize(dev)
    barrier(world)
    ev0.record()
    for _ in range(e2e_steps):
        e2e_step()
    ev1.record()
    torch.cuda.synchronize(dev)
    barrier(world)
    e2e_ms = max_over_ranks(ev0.elapsed_time(ev1), world, dev) / e2e_steps
    h2d = sum(host[k].numel() * host[k].element_size() for k in ("Qw", "K")) + \
        hV.numel() * hV.element_size()                      # the rows of V the gather reads
    d2h = sum(t.numel() * t.element_size() for t in (hK, hV, hI))
    e2e = {"value": world * tokens_per_step / (e2e_ms * 1e-3), "unit": UNIT,
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms,
           "steps": e2e_steps}

    if rank != 0:
        return
    # ---- the oracle on the host cores, bounded sample ----
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        times, cores = time_oracle(cfg, inp, 3)
        t = sum(times) / len(times)
        cpu = {"value": tokens_per_step / t, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"one full layer of {cfg.name} (all {cfg.n_kv_heads} KV heads), "
                         f"mean of 3 runs, {t:.2f} s each"}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
            "config": config_dict(cfg, {"l2": f"rotating {ROTATING_SETS} resident input sets "
                                              f"({ROTATING_SETS * 67} MB of K) > 126 MB L2"}),
            "roofline": roofline, "cpu_baseline": cpu, "clocks": clocks.summary(), "e2e": e2e,
            "gpu_launches": int(launches)}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="llama31_8b_32k", choices=list(wl.CONFIGS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    cfg = wl.CONFIGS[args.workload]
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)
    if int(os.environ.get("WORLD_SIZE", "1")) > 1 and args.impl == "ours":
        import torch.distributed as dist
        if dist.is_initialized():
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
