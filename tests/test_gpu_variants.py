"""GPU parity of the variants around the default path: KNorm as the initial score, the enhanced
and evicted signals, average pooling, value-to-value and key-to-value edges, and re-picking the
sources every round.  Same procedure as the main parity tests: discrete decisions are compared
with teacher forcing on the GPU's own fp32 values, arithmetic within the score tolerance."""
import numpy as np
import pytest
import torch

from oracle import graphkv_oracle as okv
from paper_2509_00388_b200 import workloads as wl
from tests import parity_util as pu

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def gk():
    from paper_2509_00388_b200 import binding
    binding.lib()
    return binding


def small_cfg(**kw):
    base = dict(n_prefix=5300, budget=300, n_q_heads=8, n_kv_heads=2, n_clusters=32, neighbors=8)
    base.update(kw)
    return wl.scaled(wl.LLAMA_32K, **base)


def kwargs(cfg, **extra):
    d = dict(window=cfg.window, budget=cfg.budget, pool_kernel=cfg.pool_kernel,
             topk_nodes=cfg.topk_nodes, neighbors=cfg.neighbors, rounds=cfg.rounds, decay=cfg.decay)
    d.update(extra)
    return d


@pytest.mark.parametrize("head_dim", [128, 64])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_knorm_scores_and_the_path_behind_them(gk, dtype, head_dim):
    cfg = small_cfg(dtype=dtype, head_dim=head_dim,
                    n_prefix=4500 if dtype == "bf16" and head_dim == 128 else 1800)
    inp = wl.make_inputs(cfg)
    Kd, Vd = inp["K"].to(DEV), inp["V"].to(DEV)
    kw = kwargs(cfg)
    p = gk.make_params(Kd, V=Vd, n_q_heads=cfg.n_q_heads, **kw)
    ws = gk.alloc_workspace(p, DEV)
    K_out, V_out, idx, s = gk.alloc_outputs(p, Kd)
    gk.graphkv_score_knorm(p, Kd, s)
    s0 = s.cpu()
    assert pu.score_rel_err(s0, okv.score_knorm(inp["K"], cfg.window)) <= 1e-5
    src = torch.empty((1, 2, cfg.topk_nodes), dtype=torch.int32, device=DEV)
    gk.graphkv_propagate(p, Kd, s, src, ws)
    gk.graphkv_select_gather(p, s, Kd, Vd, K_out, V_out, idx, ws)
    assert gk.graphkv_read_status(ws) == gk.OK
    n = cfg.n_prefix
    for h in range(2):
        want_src = okv.topk(s0[0, h], cfg.topk_nodes)
        assert sorted(src[0, h].tolist()) == sorted(want_src.tolist())
        o_s, *_ = okv.propagate_unit(inp["K"][0, h], s0[0, h], n, cfg.topk_nodes, cfg.neighbors,
                                     cfg.rounds, cfg.decay)
        assert pu.score_rel_err(s.cpu()[0, h][None], o_s[None]) <= pu.SCORE_RTOL
        want_idx = np.sort(okv.topk(s.cpu()[0, h], cfg.budget).numpy())
        assert np.array_equal(idx.cpu()[0, h].numpy(), want_idx)


@pytest.mark.parametrize("signal", [1, 2])
@pytest.mark.parametrize("env_simt", [False, True])
def test_enhanced_and_evicted_signals(gk, signal, env_simt, monkeypatch):
    if env_simt:
        monkeypatch.setenv("GRAPHKV_FORCE_SIMT", "1")
        monkeypatch.setenv("GRAPHKV_NO_CLUSTER", "1")
    cfg = small_cfg(rounds=2, decay=0.5)
    inp = wl.make_inputs(cfg)
    Qd, Kd, Vd = (inp[k].to(DEV) for k in ("Qw", "K", "V"))
    kw = kwargs(cfg, signal=signal)
    p = gk.make_params(Kd, Qw=Qd, V=Vd, **kw)
    ws = gk.alloc_workspace(p, DEV)
    K_out, V_out, idx, s = gk.alloc_outputs(p, Kd)
    gk.graphkv_score(p, Qd, Kd, s, ws)
    s0 = s.cpu()
    src = torch.empty((1, 2, cfg.topk_nodes), dtype=torch.int32, device=DEV)
    gk.graphkv_propagate(p, Kd, s, src, ws)
    nbr = torch.empty((1, 2, cfg.topk_nodes, cfg.neighbors), dtype=torch.int32, device=DEV)
    gk.graphkv_read_neighbors(p, ws, nbr, None)
    s1 = s.cpu()
    # the fused call gives the same bytes
    K2, V2, idx2, s2 = gk.alloc_outputs(p, Kd)
    gk.graphkv_compress(p, Qd, Kd, Vd, K2, V2, idx2, s2, ws)
    assert gk.graphkv_read_status(ws) == gk.OK
    assert torch.equal(s2.cpu().view(torch.int32), s1.view(torch.int32))
    n = cfg.n_prefix
    for h in range(2):
        o_s, *_ = okv.propagate_unit(inp["K"][0, h], s0[0, h], n, cfg.topk_nodes, cfg.neighbors,
                                     cfg.rounds, cfg.decay, forced_src=src.cpu()[0, h],
                                     forced_nbr=nbr.cpu()[0, h], signal=signal)
        g, o = s1[0, h].numpy(), o_s.numpy()
        assert np.array_equal(np.isinf(g), np.isinf(o))
        fin = np.isfinite(o)
        assert pu.score_rel_err(torch.from_numpy(g[fin])[None], torch.from_numpy(o[fin])[None]) <= pu.SCORE_RTOL
        if signal == 1:
            assert np.all(g >= s0[0, h].numpy())
        else:
            assert set(np.flatnonzero(np.isinf(g)).tolist()) == set(nbr.cpu()[0, h].reshape(-1).tolist())
        want_idx = np.sort(okv.topk(s1[0, h], cfg.budget).numpy())
        assert np.array_equal(idx2.cpu()[0, h].numpy(), want_idx)


@pytest.mark.parametrize("env_simt", [False, True])
def test_average_pooling(gk, env_simt, monkeypatch):
    if env_simt:
        monkeypatch.setenv("GRAPHKV_NO_CLUSTER", "1")
    cfg = small_cfg(pool_kernel=5)
    inp = wl.make_inputs(cfg)
    Qd, Kd, Vd = (inp[k].to(DEV) for k in ("Qw", "K", "V"))
    kw = kwargs(cfg, pool_mode=gk.POOL_AVG)
    p = gk.make_params(Kd, Qw=Qd, V=Vd, **kw)
    ws = gk.alloc_workspace(p, DEV)
    K_out, V_out, idx, s = gk.alloc_outputs(p, Kd)
    gk.graphkv_score(p, Qd, Kd, s, ws)
    s0 = s.cpu()
    assert pu.score_rel_err(s0, okv.score(inp["Qw"], inp["K"], cfg.window, 5, pool_mode=okv.POOL_AVG)) \
        <= pu.SCORE_RTOL
    src = torch.empty((1, 2, cfg.topk_nodes), dtype=torch.int32, device=DEV)
    gk.graphkv_propagate(p, Kd, s, src, ws)
    for h in range(2):
        assert sorted(src.cpu()[0, h].tolist()) == sorted(okv.topk(s0[0, h], cfg.topk_nodes).tolist())
    K2, V2, idx2, s2 = gk.alloc_outputs(p, Kd)
    gk.graphkv_compress(p, Qd, Kd, Vd, K2, V2, idx2, s2, ws)
    assert gk.graphkv_read_status(ws) == gk.OK
    assert torch.equal(s2.cpu().view(torch.int32), s.cpu().view(torch.int32))


@pytest.mark.parametrize("kinds", [("V", "V"), ("K", "V"), ("Q", "K"), ("K", "Q")])
@pytest.mark.parametrize("env_simt", [False, True])
def test_value_edges(gk, kinds, env_simt, monkeypatch):
    if env_simt:
        monkeypatch.setenv("GRAPHKV_FORCE_SIMT", "1")
    cfg = small_cfg()
    inp = wl.make_inputs(cfg)
    if "Q" in kinds:
        # query-to-key edges: the caller hands the per-KV-head query vectors of every token in the
        # argument named V (a second draw of the key recipe stands in for them here)
        inp["V"] = wl.make_inputs(cfg, layer=1)["K"]
        kinds = tuple("V" if k == "Q" else k for k in kinds)
    Qd, Kd, Vd = (inp[k].to(DEV) for k in ("Qw", "K", "V"))
    kw = kwargs(cfg)
    p = gk.make_params(Kd, Qw=Qd, V=Vd, **kw)
    ws = gk.alloc_workspace(p, DEV)
    _, _, _, s = gk.alloc_outputs(p, Kd)
    gk.graphkv_score(p, Qd, Kd, s, ws)
    s0 = s.cpu()
    src = torch.empty((1, 2, cfg.topk_nodes), dtype=torch.int32, device=DEV)
    code = {"K": gk.TENSOR_K, "V": gk.TENSOR_V}
    gk.graphkv_propagate_edges(p, Kd, Vd, code[kinds[0]], code[kinds[1]], s, src, ws)
    nbr = torch.empty((1, 2, cfg.topk_nodes, cfg.neighbors), dtype=torch.int32, device=DEV)
    nbr_e = torch.empty(nbr.shape, dtype=torch.float32, device=DEV)
    gk.graphkv_read_neighbors(p, ws, nbr, nbr_e)
    assert gk.graphkv_read_status(ws) == gk.OK
    n = cfg.n_prefix
    rep = pu.Report()
    for h in range(2):
        S, A = inp[kinds[0]][0, h], inp[kinds[1]][0, h]
        g_src = src.cpu()[0, h].numpy()
        for a, i in enumerate(g_src.tolist()):
            e = okv.edges_unit(A, n, i, Sh=S).numpy()
            got = nbr.cpu()[0, h, a].numpy()
            assert np.abs(nbr_e.cpu()[0, h, a].double().numpy() - e[got]).max() <= pu.EDGE_TIE
            want = okv.topk(torch.from_numpy(e.astype(np.float32)), cfg.neighbors, skip=i).numpy()
            diff = set(got.tolist()) ^ set(want.tolist())
            assert all(abs(e[j] - e[want].min()) <= pu.EDGE_TIE for j in diff)
        o_s, *_ = okv.propagate_unit(A, s0[0, h], n, cfg.topk_nodes, cfg.neighbors, cfg.rounds, cfg.decay,
                                     forced_src=src.cpu()[0, h], forced_nbr=nbr.cpu()[0, h], Sh=S)
        assert pu.score_rel_err(s.cpu()[0, h][None], o_s[None]) <= pu.SCORE_RTOL


@pytest.mark.parametrize("env_simt", [False, True])
def test_reselecting_sources_every_round(gk, env_simt, monkeypatch):
    if env_simt:
        monkeypatch.setenv("GRAPHKV_FORCE_SIMT", "1")
    # exact copies of keys: a source's copies score like it, are its nearest neighbours and lose
    # nine tenths of their score in the first round, so the next round has to pick other sources
    # (decay below 1: at cosine 1 a factor 1 - e carries the fp32 error of e in full)
    cfg = small_cfg(rounds=3, decay=0.9, dup_frac=0.5, dup_sigma=0.0, pool_kernel=1)
    inp = wl.make_inputs(cfg)
    Qd, Kd, Vd = (inp[k].to(DEV) for k in ("Qw", "K", "V"))
    p = gk.make_params(Kd, Qw=Qd, V=Vd, **kwargs(cfg, reselect=1))
    p1 = gk.make_params(Kd, Qw=Qd, V=Vd, **kwargs(cfg, rounds=1))
    ws = gk.alloc_workspace(p, DEV)
    K_out, V_out, idx, s = gk.alloc_outputs(p, Kd)
    gk.graphkv_score(p, Qd, Kd, s, ws)
    s_round = s.clone()
    gk.graphkv_propagate(p, Kd, s, None, ws)
    # the same as T single-round calls, each compared with the oracle's single round from the
    # GPU's scores (sources exact on the fp32 scores, neighbourhoods valid, arithmetic in tolerance)
    n = cfg.n_prefix
    src = torch.empty((1, 2, cfg.topk_nodes), dtype=torch.int32, device=DEV)
    nbr = torch.empty((1, 2, cfg.topk_nodes, cfg.neighbors), dtype=torch.int32, device=DEV)
    nbr_e = torch.empty(nbr.shape, dtype=torch.float32, device=DEV)
    seen = []
    for t in range(cfg.rounds):
        before = s_round.cpu()
        gk.graphkv_propagate(p1, Kd, s_round, src, ws)
        gk.graphkv_read_neighbors(p1, ws, nbr, nbr_e)
        seen.append(sorted(src.cpu()[0, 0].tolist()))
        rep = pu.Report()
        for h in range(2):
            assert sorted(src.cpu()[0, h].tolist()) == sorted(okv.topk(before[0, h], cfg.topk_nodes).tolist())
            pu.check_neighbourhoods(inp["K"][0, h], n, cfg.neighbors, src.cpu()[0, h].numpy(),
                                    nbr.cpu()[0, h].numpy(), nbr_e.cpu()[0, h].numpy(), rep, f"round {t} h={h}")
            o_s, *_ = okv.propagate_unit(inp["K"][0, h], before[0, h], n, cfg.topk_nodes, cfg.neighbors, 1,
                                         cfg.decay, forced_src=src.cpu()[0, h], forced_nbr=nbr.cpu()[0, h])
            assert pu.score_rel_err(s_round.cpu()[0, h][None], o_s[None]) <= pu.SCORE_RTOL
    assert torch.equal(s.cpu().view(torch.int32), s_round.cpu().view(torch.int32))
    assert any(x != seen[0] for x in seen[1:]), "the sources never changed: the case tests nothing"
    # fused call, and the free-running oracle for the kept set
    K2, V2, idx2, s2 = gk.alloc_outputs(p, Kd)
    gk.graphkv_compress(p, Qd, Kd, Vd, K2, V2, idx2, s2, ws)
    assert gk.graphkv_read_status(ws) == gk.OK
    assert torch.equal(s2.cpu().view(torch.int32), s.cpu().view(torch.int32))
    for h in range(2):
        want_idx = np.sort(okv.topk(s2.cpu()[0, h], cfg.budget).numpy())
        assert np.array_equal(idx2.cpu()[0, h].numpy(), want_idx)
    _, _, o_idx, _ = okv.compress(inp["Qw"], inp["K"], inp["V"], reselect=1, **kwargs(cfg))
    common = sum(len(set(o_idx[0, h].tolist()) & set(idx2.cpu()[0, h].tolist())) for h in range(2))
    assert common >= 0.99 * 2 * cfg.budget


def test_layers_with_their_own_budgets_in_one_call(gk):
    # three layers stacked along the batch dimension, PyramidKV-style budgets; every layer must get
    # exactly what a call of its own with its budget gives
    cfg = small_cfg(batch=3, n_prefix=4200)
    inp = wl.make_inputs(cfg)
    Qd, Kd, Vd = (inp[k].to(DEV) for k in ("Qw", "K", "V"))
    budgets = [300, 170, 64]
    p = gk.make_params(Kd, Qw=Qd, V=Vd, **kwargs(cfg, budget=max(budgets)))
    ws = gk.alloc_workspace(p, DEV)
    K_out, V_out, idx, s = gk.alloc_outputs(p, Kd)
    K_out.zero_(); V_out.zero_(); idx.fill_(-1)
    gk.graphkv_compress_layers(p, budgets, Qd, Kd, Vd, K_out, V_out, idx, s, ws)
    assert gk.graphkv_read_status(ws) == gk.OK
    n = cfg.n_prefix
    for i, b in enumerate(budgets):
        # a call of its own for the layer: the same scores up to the rounding order of the sweeps'
        # partial sums (their chunking depends on how many units a call holds)
        pi = gk.make_params(Kd[i:i + 1], Qw=Qd[i:i + 1], V=Vd[i:i + 1], **kwargs(cfg, budget=b))
        wsi = gk.alloc_workspace(pi, DEV)
        Ko, Vo, io, so = gk.alloc_outputs(pi, Kd)
        gk.graphkv_compress(pi, Qd[i:i + 1], Kd[i:i + 1], Vd[i:i + 1], Ko, Vo, io, so, wsi)
        assert gk.graphkv_read_status(wsi) == gk.OK
        assert pu.score_rel_err(s[i].cpu(), so[0].cpu()) <= 1e-5
        rows = b + cfg.window
        for h in range(cfg.n_kv_heads):
            # the layer's own budget, selected exactly on the call's own scores; rows gathered bit for bit
            want = np.sort(okv.topk(s[i, h].cpu(), b).numpy())
            assert np.array_equal(idx[i, h, :b].cpu().numpy(), want)
            ii = torch.from_numpy(want).long()
            for out, X in ((K_out, inp["K"]), (V_out, inp["V"])):
                ref = torch.cat([X[i, h, ii], X[i, h, n:]])
                assert torch.equal(out[i, h, :rows].cpu().view(torch.int16), ref.view(torch.int16))
        assert torch.all(idx[i, :, b:] == -1)
        assert torch.all(K_out[i, :, rows:] == 0) and torch.all(V_out[i, :, rows:] == 0)
        overlap = sum(len(set(idx[i, h, :b].tolist()) & set(io[0, h].tolist())) for h in range(cfg.n_kv_heads))
        assert overlap >= 0.99 * b * cfg.n_kv_heads
    bad = gk.lib().graphkv_compress_layers
    import ctypes as C
    arr = (C.c_int32 * 3)(300, 301, 64)
    assert bad(C.byref(p), arr, Qd.data_ptr(), Kd.data_ptr(), Vd.data_ptr(), K_out.data_ptr(),
               V_out.data_ptr(), idx.data_ptr(), None, ws.data_ptr(), ws.numel(), None) == gk.ERR_INVALID_ARG


@pytest.mark.parametrize("dtype,rows,hq,hkv,batch", [("bf16", 5000, 8, 2, 1), ("bf16", 37, 4, 4, 2),
                                                     ("f32", 1300, 8, 1, 1), ("bf16", 544, 32, 8, 1)])
def test_decode_attention_over_a_cache(gk, dtype, rows, hq, hkv, batch):
    # one decoding step's attention over a cache of `rows` rows against the fp64 oracle
    cfg = small_cfg(dtype=dtype, n_prefix=rows - 32, n_q_heads=hq, n_kv_heads=hkv, batch=batch)
    inp = wl.make_inputs(cfg)
    K, V = inp["K"], inp["V"]
    q = inp["Qw"][:, :, -1].contiguous()                  # the last window query of every head
    want = okv.decode_attention(q, K, V)
    qd, Kd, Vd = q.to(DEV), K.to(DEV), V.to(DEV)
    p = gk.decode_params(qd, Kd, Vd)
    ws = gk.decode_workspace(p, DEV)
    out = torch.empty((batch, hq, 128), dtype=torch.float32, device=DEV)
    gk.graphkv_decode_attention(p, qd, Kd, Vd, out, ws)
    torch.cuda.synchronize()
    err = (out.cpu().double() - want).abs().max().item()
    assert err <= 2e-3 * max(want.abs().max().item(), 1e-6), err
