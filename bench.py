#!/usr/bin/env python
"""Benchmark of the GraphKV prefill-compression path on B200.

One step = one call of `graphkv_compress` (scores -> graph -> decay rounds -> top-B -> gather)
on one layer of the Llama-3.1-8B-shaped workload (32 query / 8 KV heads, head_dim 128,
N = 32768 prefix tokens, window 32, budget 512, 16 source nodes, 2 rounds), bf16, synthetic
seeded inputs.  Metric: context tokens per second per layer, all heads (batch * N / step time).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

The timed region is R blocks of K steps back to back, each block bracketed by CUDA events on the
launching stream; the step time is the median block divided by K (minimum, maximum and the SM
clock sampled during the region are reported beside it).  The default run also times the
131072-token, 4-sequence workload the same way and attaches it as `secondary`.  Workloads with
several layers (32-layer models, per-layer budgets) step through their layers in order: a step is
one layer, and the whole-model time is reported too.

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
L2_BYTES = 126e6
FALLBACK_HBM_GBS = 6650.0
SECONDARY = "long_128k_batch4"


def cfg_kwargs(cfg, layer=0):
    return dict(window=cfg.window, budget=cfg.layer_budget(layer), pool_kernel=cfg.pool_kernel,
                topk_nodes=cfg.topk_nodes, neighbors=cfg.neighbors, rounds=cfg.rounds,
                decay=cfg.decay)


def config_dict(cfg, extra=None):
    d = {"workload": cfg.name, "batch": cfg.batch, "n_layers": cfg.n_layers,
         "n_q_heads": cfg.n_q_heads, "n_kv_heads": cfg.n_kv_heads, "head_dim": cfg.head_dim,
         "n_prefix": cfg.n_prefix, "window": cfg.window, "budget": cfg.budget,
         "budget_last": cfg.budget_last, "pool_kernel": cfg.pool_kernel,
         "topk_nodes": cfg.topk_nodes, "neighbors": cfg.neighbors, "rounds": cfg.rounds,
         "decay": cfg.decay, "parallelism": "replicas"}
    if extra:
        d.update(extra)
    return d


# ---- algorithmic bytes -------------------------------------------------------------------------
def mean_budget(cfg) -> float:
    return sum(cfg.layer_budget(l) for l in range(cfg.n_layers)) / cfg.n_layers


def algorithmic_bytes(cfg, kernel: str) -> float:
    """Bytes a kernel must move per launch for one layer of cfg (inputs it has to read once and
    outputs it has to write once; on-chip intermediates are not counted)."""
    e = 2 if cfg.dtype == "bf16" else 4
    units = cfg.batch * cfg.n_kv_heads
    N, L, D, W = cfg.n_prefix, cfg.seq_len, cfg.head_dim, cfg.window
    B, Ks = mean_budget(cfg), cfg.topk_nodes
    m = cfg.neighbors
    k_sweep = units * L * D * e
    q_bytes = cfg.batch * cfg.n_q_heads * W * D * e
    row = 4 * units * N
    table = {
        "score_fused": k_sweep + q_bytes + row,
        "score_stats": k_sweep + q_bytes,
        "score_emit": units * N * D * e + q_bytes + row,
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


# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum), one ncu capture per
# kernel inside a running step (caches as the steps before left them); see
# profiles/kernels_llama31_8b_32k_ncu_warm.md.  Only for the workload and kernels those captures
# cover and only while the kernels are the ones captured; anything else reports null.
NCU_TRAFFIC = {"llama31_8b_32k": {"score_fused_tc": 73.05e6, "pool_select_sources": 0.27e6,
                                  "similarity_tc": 0.41e6, "decay_select_gather": 1.66e6}}


def path_bytes(cfg) -> float:
    """Algorithmic bytes of the whole path per layer: two sweeps of K (sources depend on all
    scores), the window queries, three passes over the fp32 score rows, the K/V gather."""
    e = 2 if cfg.dtype == "bf16" else 4
    units = cfg.batch * cfg.n_kv_heads
    return float(2 * units * cfg.seq_len * cfg.head_dim * e
                 + cfg.batch * cfg.n_q_heads * cfg.window * cfg.head_dim * e
                 + 12 * units * cfg.n_prefix
                 + 4 * units * (mean_budget(cfg) + cfg.window) * cfg.head_dim * e)


def one_sweep_bytes(cfg) -> float:
    """The stricter model: as if the second sweep of K were served on chip."""
    e = 2 if cfg.dtype == "bf16" else 4
    return path_bytes(cfg) - cfg.batch * cfg.n_kv_heads * cfg.seq_len * cfg.head_dim * e


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
                "samples": len(s), "sm_mhz_min": s[0]}


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
def input_stats(cfg, inp):
    """Sanity statistics of a generated input (first sequence, first KV head): the mean cosine of
    the keys to their head's mean direction, the share of near-duplicate pairs among 4096 sampled
    neighbours-in-position, and the query norm; a degenerate generator shows up here."""
    K = inp["K"][0, 0, :min(cfg.n_prefix, 4096)].float()
    Kn = K / K.norm(dim=1, keepdim=True).clamp_min(1e-12)
    g = Kn @ Kn[:256].T
    return {"key_norm_mean": float(K.norm(dim=1).mean()),
            "cos_mean_to_first_256": float(g.mean()),
            "cos_above_0.99_share": float((g > 0.99).float().mean()),
            "query_norm_mean": float(inp["Qw"][0, 0].float().norm(dim=1).mean())}


def measure(cfg, gk, dev, world, local, steps, warmup, blocks, with_e2e, stacked=False):
    """Times cfg on the current device.  Returns a dict of raw measurements.  With `stacked` the
    layers of a multi-layer workload sit in one allocation and one graphkv_compress_layers call
    takes them all (a step is still one layer: the call's time over the layer count)."""
    if stacked and cfg.n_layers > 1:
        return measure_stacked(cfg, gk, dev, world, local, steps, warmup, blocks)
    n_sets_layers = min(cfg.n_layers, 4)          # distinct layers' inputs generated (the rest reuse them)
    k_bytes = cfg.batch * cfg.n_kv_heads * cfg.seq_len * cfg.head_dim * (2 if cfg.dtype == "bf16" else 4)
    # distinct device copies of the inputs, so that the first sweep of a step reads HBM: enough
    # for the keys touched between two uses of a copy to exceed twice the L2
    copies = max(1, -(-int(2.0 * L2_BYTES) // (k_bytes * n_sets_layers)))
    host_sets = [wl.make_inputs(cfg, layer=l) for l in range(n_sets_layers)]
    stats = input_stats(cfg, host_sets[0])
    host = [{k: v.pin_memory() for k, v in h.items()} for h in host_sets]
    sets = [{k: v.to(dev).clone() for k, v in h.items()} for _ in range(copies) for h in host]
    params = [gk.make_params(sets[0]["K"], Qw=sets[0]["Qw"], V=sets[0]["V"], **cfg_kwargs(cfg, l))
              for l in range(cfg.n_layers)]
    ws = gk.alloc_workspace(max(params, key=gk.workspace_bytes), dev)
    bufs = {}                                     # outputs are dense per budget
    for p in params:
        if p.budget not in bufs:
            bufs[p.budget] = gk.alloc_outputs(p, sets[0]["K"], want_scores=False)[:3]
    torch.cuda.synchronize(dev)

    def step(i):
        layer = i % cfg.n_layers
        s = sets[((i // cfg.n_layers) % copies) * n_sets_layers + layer % n_sets_layers]
        p = params[layer]
        ko, vo, io = bufs[p.budget]
        gk.graphkv_compress(p, s["Qw"], s["K"], s["V"], ko, vo, io, None, ws)

    for i in range(warmup):
        step(i)
    torch.cuda.synchronize(dev)
    assert gk.graphkv_read_status(ws) == gk.OK

    # ---- timed region: `blocks` blocks of `steps` steps, inputs resident in HBM ----
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(blocks + 1)]
    launches0 = gk.graphkv_launch_count()
    barrier(world)
    torch.cuda.synchronize(dev)
    with ClockSampler(visible_gpu_index(local)) as clocks:
        evs[0].record()
        for b in range(blocks):
            for i in range(steps):
                step(b * steps + i)
            evs[b + 1].record()
        torch.cuda.synchronize(dev)
    barrier(world)
    launches = gk.graphkv_launch_count() - launches0
    per_block = sorted(evs[b].elapsed_time(evs[b + 1]) / steps for b in range(blocks))
    med = per_block[len(per_block) // 2]
    res = {"ms_per_step": max_over_ranks(med, world, dev), "ms_min": per_block[0], "ms_max": per_block[-1],
           "blocks": blocks, "launches": int(launches), "clocks": clocks.summary(),
           "input_stats": stats, "copies": copies * n_sets_layers, "k_bytes": k_bytes}

    # ---- the same steps on one input set only (its keys stay in L2 as far as they fit) ----
    if copies > 1:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for i in range(cfg.n_layers):
            step(i)
        e0.record()
        for i in range(steps):
            step(i % cfg.n_layers)
        e1.record()
        torch.cuda.synchronize(dev)
        res["ms_same_inputs"] = e0.elapsed_time(e1) / steps

    # ---- per-kernel durations: `steps` steps again with event pairs around every launch ----
    gk.graphkv_trace_enable(True)
    for i in range(steps):
        step(i)
    torch.cuda.synchronize(dev)
    gk.graphkv_trace_enable(False)
    per_kernel = defaultdict(list)
    for name, ms in gk.graphkv_trace_read(steps * 32 + 64):
        per_kernel[name].append(ms)
    res["kernels"] = {n: {"launches_per_step": len(v) / steps, "avg_ms": sum(v) / len(v),
                          "ms_per_step": sum(v) / steps} for n, v in per_kernel.items()}

    if with_e2e:
        # ---- end to end: host buffers in, compact cache out, copies inside the timed region ----
        e2e_steps = max(3, min(steps, 50))
        p = params[0]
        ko, vo, io = bufs[p.budget]
        hK = torch.empty(ko.shape, dtype=ko.dtype).pin_memory()
        hV = torch.empty(vo.shape, dtype=vo.dtype).pin_memory()
        hI = torch.empty(io.shape, dtype=io.dtype).pin_memory()
        dst, src = sets[0], host[0]

        # Qw and K are copied to the device (the sweeps read K three times); V stays in pinned host
        # memory and the gather reads its B+W kept rows per head through the mapping; the compact
        # cache and the indices are written to pinned host memory by the gather itself.
        def e2e_step():
            for k in ("Qw", "K"):
                dst[k].copy_(src[k], non_blocking=True)
            gk.graphkv_compress(p, dst["Qw"], dst["K"], src["V"], hK, hV, hI, None, ws)

        for _ in range(2):
            e2e_step()
        torch.cuda.synchronize(dev)
        barrier(world)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for _ in range(e2e_steps):
            e2e_step()
        ev1.record()
        torch.cuda.synchronize(dev)
        barrier(world)
        e2e_ms = max_over_ranks(ev0.elapsed_time(ev1), world, dev) / e2e_steps
        h2d = sum(src[k].numel() * src[k].element_size() for k in ("Qw", "K")) + \
            hV.numel() * hV.element_size()                      # the rows of V the gather reads
        d2h = sum(t.numel() * t.element_size() for t in (hK, hV, hI))
        res["e2e"] = {"value": world * cfg.batch * cfg.n_prefix / (e2e_ms * 1e-3), "unit": UNIT,
                      "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms,
                      "steps": e2e_steps}
    res["host_inputs"] = host_sets[0]
    return res


def measure_stacked(cfg, gk, dev, world, local, steps, warmup, blocks):
    n_gen = min(cfg.n_layers, 4)
    host_sets = [wl.make_inputs(cfg, layer=l) for l in range(n_gen)]
    stats = input_stats(cfg, host_sets[0])
    stack = {k: torch.cat([host_sets[l % n_gen][k] for l in range(cfg.n_layers)], dim=0).to(dev)
             for k in ("Qw", "K", "V")}
    budgets = [cfg.layer_budget(l) for l in range(cfg.n_layers)]
    kw = cfg_kwargs(cfg)
    kw["budget"] = max(budgets)
    p = gk.make_params(stack["K"], Qw=stack["Qw"], V=stack["V"], **kw)
    ws = gk.alloc_workspace(p, dev)
    ko, vo, io, _ = gk.alloc_outputs(p, stack["K"], want_scores=False)
    calls = max(1, steps // cfg.n_layers)

    def call():
        gk.graphkv_compress_layers(p, budgets, stack["Qw"], stack["K"], stack["V"], ko, vo, io, None, ws)

    for _ in range(max(3, warmup // cfg.n_layers)):
        call()
    torch.cuda.synchronize(dev)
    assert gk.graphkv_read_status(ws) == gk.OK
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(blocks + 1)]
    launches0 = gk.graphkv_launch_count()
    barrier(world)
    torch.cuda.synchronize(dev)
    with ClockSampler(visible_gpu_index(local)) as clocks:
        evs[0].record()
        for b in range(blocks):
            for _ in range(calls):
                call()
            evs[b + 1].record()
        torch.cuda.synchronize(dev)
    barrier(world)
    launches = gk.graphkv_launch_count() - launches0
    per_block = sorted(evs[b].elapsed_time(evs[b + 1]) / (calls * cfg.n_layers) for b in range(blocks))
    med = per_block[len(per_block) // 2]
    k_bytes = cfg.n_layers * cfg.n_kv_heads * cfg.seq_len * cfg.head_dim * 2
    res = {"ms_per_step": max_over_ranks(med, world, dev), "ms_min": per_block[0], "ms_max": per_block[-1],
           "blocks": blocks, "launches": int(launches), "clocks": clocks.summary(),
           "input_stats": stats, "copies": 1, "k_bytes": k_bytes}
    gk.graphkv_trace_enable(True)
    for _ in range(calls):
        call()
    torch.cuda.synchronize(dev)
    gk.graphkv_trace_enable(False)
    per_kernel = defaultdict(list)
    for name, ms in gk.graphkv_trace_read(calls * 64 + 64):
        per_kernel[name].append(ms)
    n_steps = calls * cfg.n_layers
    # per layer: a launch covers all layers, so its time and its bytes are divided alike
    res["kernels"] = {n: {"launches_per_step": len(v) / n_steps, "avg_ms": sum(v) / len(v) / cfg.n_layers,
                          "ms_per_step": sum(v) / n_steps} for n, v in per_kernel.items()}
    res["host_inputs"] = host_sets[0]
    res["e2e"] = None
    return res


def measure_decode(cfg, gk, dev, inp, peak):
    """Decode-side micro-benchmark: one decoding step's attention over the full cache of the layer
    and over the compact cache graphkv_compress leaves (B + W rows), same queries."""
    Kd, Vd, Qd = inp["K"].to(dev), inp["V"].to(dev), inp["Qw"].to(dev)
    p = gk.make_params(Kd, Qw=Qd, V=Vd, **cfg_kwargs(cfg))
    ws = gk.alloc_workspace(p, dev)
    K_out, V_out, idx, _ = gk.alloc_outputs(p, Kd, want_scores=False)
    gk.graphkv_compress(p, Qd, Kd, Vd, K_out, V_out, idx, None, ws)
    q = Qd[:, :, -1].contiguous()
    out = {}
    for name, (Kc, Vc) in {"full_cache": (Kd, Vd), "compact_cache": (K_out, V_out)}.items():
        dp = gk.decode_params(q, Kc, Vc)
        dws = gk.decode_workspace(dp, dev)
        o = torch.empty((cfg.batch, cfg.n_q_heads, cfg.head_dim), dtype=torch.float32, device=dev)
        flush = torch.empty(int(2.2 * L2_BYTES), dtype=torch.uint8, device=dev)
        times = []
        for _ in range(12):
            flush.fill_(1)                                    # the cache comes from HBM every time
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            gk.graphkv_decode_attention(dp, q, Kc, Vc, o, dws)
            e1.record()
            torch.cuda.synchronize(dev)
            times.append(e0.elapsed_time(e1))
        times = sorted(times[2:])
        ms = times[len(times) // 2]
        nbytes = 2 * Kc.numel() * Kc.element_size()
        out[name] = {"rows": int(Kc.shape[2]), "ms": ms, "cache_bytes": nbytes,
                     "achieved": nbytes / (ms * 1e-3) / 1e9, "unit": "GB/s",
                     "frac": nbytes / (ms * 1e-3) / 1e9 / peak}
    # the KNorm initial score: one pass over the prefix keys
    sc = torch.empty((cfg.batch, cfg.n_kv_heads, cfg.n_prefix), dtype=torch.float32, device=dev)
    times = []
    for _ in range(12):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        gk.graphkv_score_knorm(p, Kd, sc)
        e1.record()
        torch.cuda.synchronize(dev)
        times.append(e0.elapsed_time(e1))
    ms = sorted(times[2:])[5]
    kb = cfg.batch * cfg.n_kv_heads * cfg.n_prefix * (cfg.head_dim * Kd.element_size() + 4)
    out["knorm_score"] = {"ms": ms, "bytes": kb, "achieved": kb / (ms * 1e-3) / 1e9, "unit": "GB/s",
                          "frac": kb / (ms * 1e-3) / 1e9 / peak}
    out["speedup"] = out["full_cache"]["ms"] / out["compact_cache"]["ms"]
    out["note"] = ("attention of one decoding step, all query heads of the layer; L2 flushed before every "
                   "call; median of 10")
    return out


def roofline_blocks(cfg, res, peak, peak_kind):
    """The dominant kernel's roofline entry, the whole path's, and every kernel's."""
    kernels = res["kernels"]
    ms_step = res["ms_per_step"]
    top = max(kernels, key=lambda n: kernels[n]["ms_per_step"])
    top_bytes = algorithmic_bytes(cfg, top)
    achieved = top_bytes / (kernels[top]["avg_ms"] * 1e-3) / 1e9
    traffic = NCU_TRAFFIC.get(cfg.name, {})
    roofline = {"bound": "hbm", "kernel": top, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": traffic.get(top),
                "peak_source": f"{peak_kind} copy bandwidth",
                "algorithmic_bytes_per_launch": top_bytes,
                "avg_launch_ms": kernels[top]["avg_ms"],
                "timing": "CUDA event pairs around every launch, second pass of the same steps"}
    pb, ob = path_bytes(cfg), one_sweep_bytes(cfg)
    path = {"bound": "hbm", "algorithmic_bytes_per_step": pb, "achieved": pb / (ms_step * 1e-3) / 1e9,
            "peak": peak, "unit": "GB/s", "frac": pb / (ms_step * 1e-3) / 1e9 / peak,
            "frac_of_8tbs": pb / (ms_step * 1e-3) / 1e9 / 8000.0,
            "one_sweep_model_bytes": ob, "one_sweep_model_frac": ob / (ms_step * 1e-3) / 1e9 / peak,
            "traffic": sum(traffic.values()) if traffic and set(traffic) >= set(kernels) else None,
            "ms_x_sm_mhz": ms_step * (res["clocks"].get("sm_mhz") or 0)}
    per = {n: {"ms_per_step": round(k["ms_per_step"], 5),
               "algorithmic_bytes": algorithmic_bytes(cfg, n),
               "achieved": round(algorithmic_bytes(cfg, n) / (k["avg_ms"] * 1e-3) / 1e9, 1),
               "frac": round(algorithmic_bytes(cfg, n) / (k["avg_ms"] * 1e-3) / 1e9 / peak, 4),
               "traffic": traffic.get(n)} for n, k in kernels.items()}
    return roofline, path, per


def l2_note(res):
    mb = res["k_bytes"] / 1e6
    if res["copies"] == 1:
        return f"one resident input set: its {mb:.0f} MB of K alone exceed the 126 MB L2"
    return (f"rotating {res['copies']} resident input sets ({res['copies'] * mb:.0f} MB of K) "
            f"> 126 MB L2")


def run_ours(args, cfg):
    world, rank, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the CUDA path has no CPU fallback)")
    from paper_2509_00388_b200 import binding as gk
    gk.lib()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    peak, peak_kind = measured_peak()

    res = measure(cfg, gk, dev, world, local, args.steps, args.warmup, args.blocks, True, args.stacked)
    ms_step = res["ms_per_step"]
    tokens_per_step = cfg.batch * cfg.n_prefix
    value = world * tokens_per_step / (ms_step * 1e-3)
    roofline, path, per = roofline_blocks(cfg, res, peak, peak_kind)
    inp = res.pop("host_inputs")

    decode = None
    if world == 1 and not args.no_secondary and cfg.n_layers == 1:
        decode = measure_decode(cfg, gk, dev, inp, peak)
    secondary = None
    if world == 1 and not args.no_secondary and cfg.name != SECONDARY:
        cfg2 = wl.CONFIGS[SECONDARY]
        torch.cuda.empty_cache()
        r2 = measure(cfg2, gk, dev, world, local, max(2, args.steps // 20), 3, max(5, args.blocks // 2), False)
        r2.pop("host_inputs")
        rf2, path2, per2 = roofline_blocks(cfg2, r2, peak, peak_kind)
        secondary = {"config": config_dict(cfg2, {"l2": l2_note(r2)}),
                     "ms_per_step": r2["ms_per_step"], "ms_min": r2["ms_min"], "ms_max": r2["ms_max"],
                     "blocks": r2["blocks"],
                     "value": cfg2.batch * cfg2.n_prefix / (r2["ms_per_step"] * 1e-3), "unit": UNIT,
                     "roofline": rf2, "roofline_path": path2, "roofline_kernels": per2,
                     "clocks": r2["clocks"], "gpu_launches": r2["launches"],
                     "input_stats": r2["input_stats"]}

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
    extra = {"l2": l2_note(res)}
    if cfg.n_layers > 1:
        extra["whole_model_ms"] = ms_step * cfg.n_layers
        extra["layers"] = (f"a step is one layer; the {cfg.n_layers} layers are taken by one "
                           "graphkv_compress_layers call per model pass" if args.stacked else
                           f"a step is one layer; the {cfg.n_layers} layers are stepped through in order")
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
            "config": config_dict(cfg, extra),
            "timing": {"blocks": res["blocks"], "steps_per_block": args.steps, "statistic": "median block",
                       "ms_min": res["ms_min"], "ms_max": res["ms_max"],
                       "ms_per_step_same_inputs": res.get("ms_same_inputs")},
            "roofline": roofline, "roofline_path": path, "roofline_kernels": per,
            "cpu_baseline": cpu, "clocks": res["clocks"], "e2e": res["e2e"],
            "gpu_launches": res["launches"], "input_stats": res["input_stats"],
            "decode": decode, "secondary": secondary}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--blocks", type=int, default=25, help="timed blocks of --steps steps (median reported)")
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="llama31_8b_32k", choices=list(wl.CONFIGS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true")
    ap.add_argument("--stacked", action="store_true",
                    help="multi-layer workloads: all layers in one allocation and one call per model pass")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's number of sequences")
    ap.add_argument("--topk-nodes", type=int, default=0, help="override the workload's number of source nodes")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    cfg = wl.CONFIGS[args.workload]
    if args.batch > 0:
        cfg = wl.scaled(cfg, batch=args.batch, name=f"{cfg.name}[batch={args.batch}]")
    if args.topk_nodes > 0:
        cfg = wl.scaled(cfg, topk_nodes=args.topk_nodes, name=f"{cfg.name}[topk_nodes={args.topk_nodes}]")
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
