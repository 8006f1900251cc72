"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs, stage by stage and end to end."""
import json
import os

import numpy as np
import pytest
import torch

from oracle import graphkv_oracle as okv
from paper_2509_00388_b200 import workloads as wl
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gk():
    from paper_2509_00388_b200 import binding
    binding.lib()
    return binding


def run_staged(gk, Qw, K, V, **kw):
    """score -> propagate -> select_gather on cuda:0; returns CPU copies of every stage."""
    dev = torch.device("cuda:0")
    Qd, Kd, Vd = Qw.to(dev), K.to(dev), V.to(dev)
    p = gk.make_params(Kd, Qw=Qd, V=Vd, **kw)
    ws = gk.alloc_workspace(p, dev)
    K_out, V_out, idx, s = gk.alloc_outputs(p, Kd)
    gk.graphkv_score(p, Qd, Kd, s, ws)
    out = {"scores0": s.cpu()}
    src = None
    if kw.get("topk_nodes", 0) > 0:
        src = torch.empty((p.batch, p.n_kv_heads, p.topk_nodes), dtype=torch.int32, device=dev)
    gk.graphkv_propagate(p, Kd, s, src, ws)
    if src is not None:
        out["src"] = src.cpu()
    m = gk.resolve_neighbors(p.seq_len - p.window, p.neighbors)
    if src is not None and p.rounds > 0 and m > 0:
        nbr = torch.empty((p.batch, p.n_kv_heads, p.topk_nodes, m), dtype=torch.int32, device=dev)
        nbr_e = torch.empty(nbr.shape, dtype=torch.float32, device=dev)
        gk.graphkv_read_neighbors(p, ws, nbr, nbr_e)
        out.update(nbr=nbr.cpu(), nbr_e=nbr_e.cpu())
    out["scores"] = s.cpu()
    gk.graphkv_select_gather(p, s, Kd, Vd, K_out, V_out, idx, ws)
    assert gk.graphkv_read_status(ws) == gk.OK
    out.update(idx=idx.cpu(), K_out=K_out.cpu(), V_out=V_out.cpu())
    return out


def run_fused(gk, Qw, K, V, **kw):
    dev = torch.device("cuda:0")
    Qd, Kd, Vd = Qw.to(dev), K.to(dev), V.to(dev)
    p = gk.make_params(Kd, Qw=Qd, V=Vd, **kw)
    ws = gk.alloc_workspace(p, dev)
    K_out, V_out, idx, s = gk.alloc_outputs(p, Kd)
    gk.graphkv_compress(p, Qd, Kd, Vd, K_out, V_out, idx, s, ws)
    assert gk.graphkv_read_status(ws) == gk.OK
    out = {"idx": idx.cpu(), "K_out": K_out.cpu(), "V_out": V_out.cpu(), "scores": s.cpu()}
    m = gk.resolve_neighbors(p.seq_len - p.window, p.neighbors)
    if p.topk_nodes > 0 and p.rounds > 0 and m > 0:
        nbr = torch.empty((p.batch, p.n_kv_heads, p.topk_nodes, m), dtype=torch.int32, device=dev)
        gk.graphkv_read_neighbors(p, ws, nbr, None)
        out["nbr"] = nbr.cpu()
    return out


def cfg_kwargs(cfg, layer=0):
    return dict(window=cfg.window, budget=cfg.layer_budget(layer), pool_kernel=cfg.pool_kernel,
                topk_nodes=cfg.topk_nodes, neighbors=cfg.neighbors, rounds=cfg.rounds,
                decay=cfg.decay)


def check(gk, cfg, layer=0, sequences=None, strict_overlap=True, **override):
    inp = wl.make_inputs(cfg, layer=layer, sequences=sequences)
    kw = cfg_kwargs(cfg, layer)
    kw.update(override)
    staged = run_staged(gk, inp["Qw"], inp["K"], inp["V"], **kw)
    fused = run_fused(gk, inp["Qw"], inp["K"], inp["V"], **kw)
    for name in ("idx", "K_out", "V_out", "scores"):
        assert torch.equal(staged[name].view(torch.uint8), fused[name].view(torch.uint8)), \
            f"fused compress differs from the staged calls in {name}"
    if "nbr" in fused:
        assert torch.equal(torch.sort(staged["nbr"], dim=-1).values,
                           torch.sort(fused["nbr"], dim=-1).values), \
            "fused compress built other neighbourhoods than the staged calls"
    rep = pu.check_compress(staged, inp["Qw"], inp["K"], inp["V"], strict_overlap=strict_overlap,
                            **kw)
    print(json.dumps({"config": cfg.name, "layer": layer, **rep.as_dict()}))
    if cfg == wl.CONFIGS.get(cfg.name) and not override:
        tag = cfg.name + (f"_layer{layer}" if cfg.n_layers > 1 else "") + \
            ("" if sequences is None else "_seq" + "".join(str(q) for q in sequences))
        rep.write(tag)
    return rep


# ---- config 1: the tiny fp32 single head, with the neighbour sweep ------------------------------
@pytest.mark.parametrize("m", [0, 1, 4, 16])
@pytest.mark.parametrize("lam", [1.0, 0.5, 0.25])
def test_tiny_fp32_config(gk, m, lam):
    check(gk, wl.TINY, neighbors=m, decay=lam)


# ---- reduced copies of the large configs: several tiles and a ragged tail ----------------------
SMALL = [
    dict(n_prefix=5000, budget=300, n_q_heads=8, n_kv_heads=2, neighbors=8),
    dict(n_prefix=4097, budget=64, n_q_heads=4, n_kv_heads=4, window=32, topk_nodes=5),
    dict(n_prefix=3000, budget=500, n_q_heads=8, n_kv_heads=2, window=64, topk_nodes=32, rounds=4),
    dict(n_prefix=2049, budget=100, n_q_heads=4, n_kv_heads=1, window=17, batch=3, neighbors=3),
    dict(n_prefix=1024, budget=1024, n_q_heads=2, n_kv_heads=2, window=8),
    # query rows per KV head that fill 5, 6 and 7 of the 8 accumulator slices of the score sweeps
    dict(n_prefix=3500, budget=200, n_q_heads=6, n_kv_heads=2, window=48),
    dict(n_prefix=2700, budget=150, n_q_heads=5, n_kv_heads=1, window=37, batch=2),
    dict(n_prefix=3100, budget=120, n_q_heads=7, n_kv_heads=1, window=32, topk_nodes=24),
]


@pytest.mark.parametrize("i", range(len(SMALL)))
def test_reduced_bf16_configs(gk, i):
    cfg = wl.scaled(wl.LLAMA_32K, n_clusters=32, **SMALL[i])
    check(gk, cfg, strict_overlap=False)


def test_reduced_fp32_multihead(gk):
    cfg = wl.scaled(wl.LLAMA_32K, dtype="f32", n_prefix=2500, budget=200, n_q_heads=8,
                    n_kv_heads=2, n_clusters=32, neighbors=6)
    check(gk, cfg, strict_overlap=False)


# ---- degenerate and edge cases ----------------------------------------------------------------
@pytest.mark.parametrize("case", [
    dict(n_prefix=40, budget=7, topk_nodes=3, neighbors=2),            # N below every tile size
    dict(n_prefix=1, budget=1, topk_nodes=1, neighbors=0),             # single node, m = 0
    dict(n_prefix=2, budget=1, topk_nodes=2, neighbors=1),
    dict(n_prefix=333, budget=333, topk_nodes=4, neighbors=5),         # keep everything
    dict(n_prefix=333, budget=1, topk_nodes=333, neighbors=1),         # every node a source
    dict(n_prefix=600, budget=50, topk_nodes=0, neighbors=0),          # no sources
    dict(n_prefix=600, budget=50, topk_nodes=4, neighbors=0, rounds=0),  # T = 0: base method
    dict(n_prefix=600, budget=50, topk_nodes=4, neighbors=7, pool_kernel=1),
    dict(n_prefix=600, budget=50, topk_nodes=2, neighbors=599),        # m = N - 1
    dict(n_prefix=600, budget=50, topk_nodes=4, neighbors=7, decay=0.0),
    dict(n_prefix=700, budget=50, topk_nodes=4, neighbors=7, pool_kernel=31),
])
def test_edge_cases(gk, case):
    cfg = wl.scaled(wl.LLAMA_32K, n_q_heads=4, n_kv_heads=2, n_clusters=8, **case)
    check(gk, cfg, strict_overlap=False)


def test_zero_queries_give_constant_scores_and_lowest_indices(gk):
    cfg = wl.scaled(wl.LLAMA_32K, n_prefix=3000, budget=77, n_q_heads=4, n_kv_heads=2, rounds=0)
    inp = wl.make_inputs(cfg)
    Qw = torch.zeros_like(inp["Qw"])
    out = run_fused(gk, Qw, inp["K"], inp["V"], **cfg_kwargs(cfg))
    expect = cfg.group * sum(1.0 / (cfg.n_prefix + r + 1) for r in range(cfg.window))
    assert pu.score_rel_err(out["scores"], torch.full_like(out["scores"], expect)) < 1e-5
    assert torch.equal(out["idx"], torch.arange(77, dtype=torch.int32).expand(1, 2, 77))


def test_tail_source_selection_takes_its_radix_path_on_constant_scores(gk):
    # all-zero queries make every score equal: the sources are the lowest positions, and the
    # selection at the tail of the emit sweep must reach them through its search over the pooled
    # row (its candidate lists overflow); the staged calls pick them with the pooling kernel
    cfg = wl.scaled(wl.LLAMA_32K, n_prefix=3000, budget=77, n_q_heads=4, n_kv_heads=2, rounds=1,
                    topk_nodes=16, neighbors=4)
    inp = wl.make_inputs(cfg)
    Qw = torch.zeros_like(inp["Qw"])
    kw = cfg_kwargs(cfg)
    old = os.environ.get("GRAPHKV_TAIL_SOURCES")
    os.environ["GRAPHKV_TAIL_SOURCES"] = "1"
    try:
        staged = run_staged(gk, Qw, inp["K"], inp["V"], **kw)
        fused = run_fused(gk, Qw, inp["K"], inp["V"], **kw)
    finally:
        if old is None:
            os.environ.pop("GRAPHKV_TAIL_SOURCES", None)
        else:
            os.environ["GRAPHKV_TAIL_SOURCES"] = old
    assert torch.equal(staged["src"], torch.arange(16, dtype=torch.int32).expand(1, 2, 16))
    for name in ("idx", "K_out", "V_out", "scores"):
        assert torch.equal(staged[name].view(torch.uint8), fused[name].view(torch.uint8)), name
    assert torch.equal(torch.sort(staged["nbr"], dim=-1).values, torch.sort(fused["nbr"], dim=-1).values)


def test_exact_duplicate_keys_tie_break_like_the_oracle(gk):
    # bit-identical keys give bit-identical cosines: the lower index must win on both sides
    cfg = wl.scaled(wl.LLAMA_32K, n_prefix=2000, budget=100, n_q_heads=4, n_kv_heads=1,
                    n_clusters=8, dup_sigma=0.0, dup_frac=0.5, neighbors=16)
    check(gk, cfg, strict_overlap=False)


def test_identical_keys_take_the_exact_tie_paths(gk):
    # every key of a head is the same vector: all cosines tie, so each source's neighbourhood is
    # decided by position alone (the m lowest positions other than the source itself) and the
    # candidate lists of every key chunk overflow into their exact bisection paths
    cfg = wl.scaled(wl.LLAMA_32K, n_prefix=5000, budget=200, n_q_heads=4, n_kv_heads=2,
                    n_clusters=8, topk_nodes=16, neighbors=32, rounds=1, pool_kernel=1)
    inp = wl.make_inputs(cfg)
    K = inp["K"].clone()
    K[:, :, :, :] = K[:, :, :1, :]
    kw = cfg_kwargs(cfg)
    staged = run_staged(gk, inp["Qw"], K, inp["V"], **kw)
    fused = run_fused(gk, inp["Qw"], K, inp["V"], **kw)
    for name in ("idx", "K_out", "V_out", "scores"):
        assert torch.equal(staged[name].view(torch.uint8), fused[name].view(torch.uint8))
    n = cfg.n_prefix
    for h in range(cfg.n_kv_heads):
        s0 = staged["scores0"][0, h]
        o_s, o_src, o_nbr, _ = okv.propagate_unit(K[0, h], s0, n, cfg.topk_nodes, cfg.neighbors,
                                                  cfg.rounds, cfg.decay)
        assert sorted(staged["src"][0, h].tolist()) == sorted(o_src.tolist())
        changed = set(torch.nonzero(staged["scores"][0, h] != s0).flatten().tolist())
        want = set(o_nbr.flatten().tolist())
        assert changed == {j for j in want if float(s0[j]) != 0.0}
        assert pu.score_rel_err(staged["scores"][0, h][None], o_s[None]) <= pu.SCORE_RTOL
        want_idx = np.sort(okv.topk(staged["scores"][0, h], cfg.budget).numpy())
        assert np.array_equal(staged["idx"][0, h].numpy(), want_idx)


@pytest.mark.parametrize("env", [{"GRAPHKV_NO_CLUSTER": "1"}, {"GRAPHKV_FORCE_SIMT": "1"},
                                 {"GRAPHKV_NO_CLUSTER": "1", "GRAPHKV_FORCE_SIMT": "1"},
                                 {"GRAPHKV_L2_GROUP_MB": "1"}, {"GRAPHKV_TWO_SCORE_KERNELS": "1"},
                                 {"GRAPHKV_TAIL_SOURCES": "1"},
                                 {"GRAPHKV_TAIL_SOURCES": "1", "GRAPHKV_NO_CLUSTER": "1"}])
def test_fallback_kernels_agree_with_the_oracle(gk, env):
    # the generic row kernels (rows too long for a cluster), the SIMT sweeps (fp32 inputs, many
    # sources or neighbours), several launch groups, the two score sweeps as kernels of their own
    # (launches with more CTAs than SMs), and the source selection at the tail of the
    # emit sweep with pooling in the finishing kernel, forced here on a case the fast path covers
    cfg = wl.scaled(wl.LLAMA_32K, n_prefix=4500, budget=300, n_q_heads=8, n_kv_heads=2,
                    n_clusters=32, neighbors=8, batch=2)
    old = {k: os.environ.get(k) for k in env}
    os.environ.update(env)
    try:
        check(gk, cfg, strict_overlap=False)
    finally:
        for k, v in old.items():
            if v is None:
                os.environ.pop(k, None)
            else:
                os.environ[k] = v

@pytest.mark.parametrize("window", [32, 64])
def test_one_score_kernel_and_two_agree_to_the_bit(gk, window):
    # the kernel that runs both sweeps (launches whose CTAs are all resident) and the two-kernel
    # path merge the row statistics in the same order: identical scores
    dev = torch.device("cuda:0")
    cfg = wl.scaled(wl.LLAMA_32K, n_prefix=9000 + 37, budget=128, n_q_heads=8, n_kv_heads=2,
                    n_clusters=32, window=window)
    inp = wl.make_inputs(cfg)
    Qd, Kd = inp["Qw"].to(dev), inp["K"].to(dev)
    p = gk.make_params(Kd, Qw=Qd, window=cfg.window, pool_kernel=cfg.pool_kernel)
    ws = gk.alloc_workspace(p, dev)
    one = torch.empty((p.batch, p.n_kv_heads, cfg.n_prefix), dtype=torch.float32, device=dev)
    two = torch.empty_like(one)
    gk.graphkv_score(p, Qd, Kd, one, ws)
    os.environ["GRAPHKV_TWO_SCORE_KERNELS"] = "1"
    try:
        gk.graphkv_score(p, Qd, Kd, two, ws)
    finally:
        os.environ.pop("GRAPHKV_TWO_SCORE_KERNELS", None)
    assert gk.graphkv_read_status(ws) == gk.OK
    assert torch.equal(one, two)
    want = okv.score(inp["Qw"], inp["K"], cfg.window, cfg.pool_kernel)
    assert pu.score_rel_err(one.cpu(), want) <= pu.SCORE_RTOL

@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_head_dimension_64(gk, dtype):
    # heads of 64 dimensions take the general kernels for the scores, the edges and the gather
    # (the tensor-core kernels are written for 128) and the same row kernels
    cfg = wl.scaled(wl.LLAMA_32K, head_dim=64, dtype=dtype, n_prefix=3000 + 21, budget=200, n_q_heads=8,
                    n_kv_heads=2, n_clusters=24, neighbors=8, batch=2)
    check(gk, cfg, strict_overlap=False)


@pytest.mark.parametrize("case", [
    dict(topk_nodes=40, neighbors=12),                  # source count padded to 64
    dict(topk_nodes=64, neighbors=32),                  # the largest tensor-core similarity case
    dict(topk_nodes=65, neighbors=8),                   # one more: a second sweep for one source
    dict(topk_nodes=154, neighbors=8, budget=512),      # 0.3 x budget, three sweeps of 64 sources
    dict(topk_nodes=154, neighbors=32, budget=512, rounds=1),   # lists beyond the default staging
    dict(topk_nodes=12, neighbors=33),                  # neighbours above the candidate-list path
    dict(topk_nodes=12, neighbors=8, pool_kernel=131),  # pooling halo above the cluster kernel's
    dict(topk_nodes=3, neighbors=32, rounds=5, decay=0.5),
])
def test_regime_boundaries(gk, case):
    cfg = wl.scaled(wl.LLAMA_32K, **{**dict(n_prefix=6100, budget=400, n_q_heads=8, n_kv_heads=2,
                                            n_clusters=48), **case})
    check(gk, cfg, strict_overlap=False)


def test_row_longer_than_a_cluster_holds(gk):
    # N above 8 x 32768: pooling, selections, decay and gather take the generic kernels
    cfg = wl.scaled(wl.LLAMA_32K, n_prefix=270000, budget=700, n_q_heads=1, n_kv_heads=1,
                    window=8, n_clusters=64, topk_nodes=8, neighbors=16)
    check(gk, cfg, strict_overlap=False)


def test_strided_inputs(gk):
    # K and V as views of a [batch, L, heads, D] buffer (token-major, the layout of a fused
    # QKV projection): strides are not those of a dense [b, h, L, D] tensor
    cfg = wl.scaled(wl.LLAMA_32K, n_prefix=1500, budget=100, n_q_heads=8, n_kv_heads=2,
                    n_clusters=16, batch=2)
    inp = wl.make_inputs(cfg)
    dev = torch.device("cuda:0")
    kw = cfg_kwargs(cfg)
    dense = run_fused(gk, inp["Qw"], inp["K"], inp["V"], **kw)
    Kt = inp["K"].to(dev).permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    Vt = inp["V"].to(dev).permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    Qd = inp["Qw"].to(dev)
    assert not Kt.is_contiguous()
    p = gk.make_params(Kt, Qw=Qd, V=Vt, **kw)
    ws = gk.alloc_workspace(p, dev)
    K_out, V_out, idx, s = gk.alloc_outputs(p, Kt)
    gk.graphkv_compress(p, Qd, Kt, Vt, K_out, V_out, idx, s, ws)
    assert torch.equal(idx.cpu(), dense["idx"])
    assert torch.equal(K_out.cpu().view(torch.int16), dense["K_out"].view(torch.int16))
    assert torch.equal(V_out.cpu().view(torch.int16), dense["V_out"].view(torch.int16))
    assert torch.equal(s.cpu(), dense["scores"])


def test_values_and_outputs_in_pinned_host_memory(gk):
    # V is only gathered from: it may stay in page-locked host memory (same pointer on the device
    # under unified addressing), and the compact cache may be written there directly
    cfg = wl.scaled(wl.LLAMA_32K, n_prefix=5200, budget=300, n_q_heads=8, n_kv_heads=2, batch=2)
    inp = wl.make_inputs(cfg)
    dev = torch.device("cuda:0")
    kw = cfg_kwargs(cfg)
    ref = run_fused(gk, inp["Qw"], inp["K"], inp["V"], **kw)
    Qd, Kd = inp["Qw"].to(dev), inp["K"].to(dev)
    Vh = inp["V"].pin_memory()
    p = gk.make_params(Kd, Qw=Qd, V=Vh, **kw)
    ws = gk.alloc_workspace(p, dev)
    K_out, _, idx, _ = gk.alloc_outputs(p, Kd, want_scores=False)
    V_out = torch.empty(K_out.shape, dtype=K_out.dtype).pin_memory()
    gk.graphkv_compress(p, Qd, Kd, Vh, K_out, V_out, idx, None, ws)
    assert gk.graphkv_read_status(ws) == gk.OK          # synchronises the stream
    assert torch.equal(idx.cpu(), ref["idx"])
    assert torch.equal(K_out.cpu().view(torch.int16), ref["K_out"].view(torch.int16))
    assert torch.equal(V_out.view(torch.int16), ref["V_out"].view(torch.int16))


def test_runs_are_bitwise_repeatable(gk):
    cfg = wl.scaled(wl.LLAMA_32K, n_prefix=6000, budget=256, n_q_heads=8, n_kv_heads=2)
    inp = wl.make_inputs(cfg)
    a = run_fused(gk, inp["Qw"], inp["K"], inp["V"], **cfg_kwargs(cfg))
    b = run_fused(gk, inp["Qw"], inp["K"], inp["V"], **cfg_kwargs(cfg))
    for name in a:
        assert torch.equal(a[name].view(torch.uint8), b[name].view(torch.uint8)), name


def test_select_gather_alone_is_bit_exact_with_planted_ties(gk):
    dev = torch.device("cuda:0")
    for n, B, seed in [(5000, 300, 0), (131072, 4096, 1), (33, 33, 2), (1025, 1, 3)]:
        s = wl.make_scores(3, n, seed, tie_frac=0.3).reshape(1, 3, n)
        cfg = wl.scaled(wl.LLAMA_32K, n_prefix=n, budget=B, n_q_heads=3, n_kv_heads=3, window=4)
        inp = wl.make_inputs(cfg)
        Kd, Vd = inp["K"].to(dev), inp["V"].to(dev)
        p = gk.make_params(Kd, V=Vd, window=4, budget=B)
        ws = gk.alloc_workspace(p, dev)
        K_out, V_out, idx, _ = gk.alloc_outputs(p, Kd, want_scores=False)
        gk.graphkv_select_gather(p, s.to(dev), Kd, Vd, K_out, V_out, idx, ws)
        oK, oV, oidx = okv.select_gather(s, inp["K"], inp["V"], 4, B)
        assert torch.equal(idx.cpu(), oidx)
        assert torch.equal(K_out.cpu().view(torch.int16), oK.view(torch.int16))
        assert torch.equal(V_out.cpu().view(torch.int16), oV.view(torch.int16))


def test_propagate_alone_from_oracle_scores(gk):
    # teacher forcing the other way: the GPU stage starts from the oracle's fp32 scores
    cfg = wl.scaled(wl.LLAMA_32K, n_prefix=7000, budget=256, n_q_heads=8, n_kv_heads=2,
                    n_clusters=64)
    inp = wl.make_inputs(cfg)
    s0 = okv.score(inp["Qw"], inp["K"], cfg.window, cfg.pool_kernel)
    o_s, o_src = okv.propagate(inp["K"], s0, cfg.window, cfg.topk_nodes, cfg.neighbors,
                               cfg.rounds, cfg.decay)
    dev = torch.device("cuda:0")
    Kd = inp["K"].to(dev)
    p = gk.make_params(Kd, n_q_heads=cfg.n_q_heads, **cfg_kwargs(cfg))
    ws = gk.alloc_workspace(p, dev)
    s = s0.to(dev)
    src = torch.empty((1, 2, cfg.topk_nodes), dtype=torch.int32, device=dev)
    gk.graphkv_propagate(p, Kd, s, src, ws)
    assert torch.equal(torch.sort(src.cpu(), dim=-1).values.int(),
                       torch.sort(o_src, dim=-1).values.int())
    assert pu.score_rel_err(s.cpu(), o_s) <= pu.SCORE_RTOL


# ---- the benchmark configurations at full size -------------------------------------------------
def test_full_llama_32k(gk):
    rep = check(gk, wl.LLAMA_32K)
    assert rep.overlap >= pu.MIN_OVERLAP


@pytest.mark.parametrize("layer", [0, 13, 31])
def test_full_mistral_16k_layers(gk, layer):
    check(gk, wl.MISTRAL_16K, layer=layer)


def test_full_mistral_16k_with_the_papers_source_count(gk):
    # the source count the paper's ablation finds best: 0.3 x budget = 614 sources per head
    cfg = wl.scaled(wl.MISTRAL_16K, topk_nodes=round(0.3 * wl.MISTRAL_16K.budget))
    assert cfg.topk_nodes == 614
    check(gk, cfg, layer=0)


@pytest.mark.parametrize("layer", [0, 16, 31])
def test_full_pyramid_budgets(gk, layer):
    cfg = wl.PYRAMID_32K
    assert cfg.layer_budget(0) == 2048 and cfg.layer_budget(31) == 128
    check(gk, cfg, layer=layer)


def test_full_long_context_128k(gk):
    # all four sequences of the batch, two at a time to bound host memory
    for seqs in ([0, 1], [2, 3]):
        check(gk, wl.LONG_128K, sequences=seqs)
