"""Calls on two streams at once, a workspace each: the library keeps no state outside the
workspaces, so concurrent calls must give the results of calls made one after the other.  The kernel
that runs both score sweeps makes the CTAs of a unit wait for one another; two such kernels in
flight together must not starve each other of SMs (every wait is bounded: a problem would show as
GRAPHKV_ERR_TIMEOUT, not as a hang)."""
import os

import pytest
import torch

from paper_2509_00388_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_two_streams_with_a_workspace_each_agree_with_serial_calls():
    from paper_2509_00388_b200 import binding as gk
    gk.lib()
    dev = torch.device("cuda:0")
    # eight units of 16 chunks each fill most of the machine with one call's score kernel
    cfg = wl.scaled(wl.LLAMA_32K, n_prefix=16384, budget=256)
    inp = {k: v.to(dev) for k, v in wl.make_inputs(cfg).items()}
    kw = dict(window=cfg.window, budget=cfg.budget, pool_kernel=cfg.pool_kernel, topk_nodes=cfg.topk_nodes,
              neighbors=cfg.neighbors, rounds=cfg.rounds, decay=cfg.decay)
    p = gk.make_params(inp["K"], Qw=inp["Qw"], V=inp["V"], **kw)
    ws = [gk.alloc_workspace(p, dev) for _ in range(2)]
    outs = [gk.alloc_outputs(p, inp["K"]) for _ in range(3)]

    def call(o, w):
        gk.graphkv_compress(p, inp["Qw"], inp["K"], inp["V"], o[0], o[1], o[2], o[3], w)

    call(outs[2], ws[0])
    torch.cuda.synchronize()
    assert gk.graphkv_read_status(ws[0]) == gk.OK
    streams = [torch.cuda.Stream(dev) for _ in range(2)]
    os.environ["GRAPHKV_WAIT_CYCLES"] = "200000000"          # a tenth of a second per wait
    try:
        for it in range(40):
            for q in range(2):
                with torch.cuda.stream(streams[q]):
                    call(outs[q], ws[q])
        torch.cuda.synchronize()
    finally:
        os.environ.pop("GRAPHKV_WAIT_CYCLES", None)
    for q in range(2):
        with torch.cuda.stream(streams[q]):
            assert gk.graphkv_read_status(ws[q]) == gk.OK
        for got, want in zip(outs[q], outs[2]):
            assert torch.equal(got.view(torch.uint8), want.view(torch.uint8))


@pytest.mark.parametrize("two_kernels", [False, True])
def test_a_workspace_nobody_cleared_gives_the_same_result(two_kernels):
    # the calls that start at step (I) set up every word of the workspace they rely on themselves
    # (counters tagged per call or cleared on the way), so its content before the call is irrelevant
    from paper_2509_00388_b200 import binding as gk
    gk.lib()
    dev = torch.device("cuda:0")
    cfg = wl.scaled(wl.LLAMA_32K, n_prefix=6000 + 13, budget=200, n_q_heads=8, n_kv_heads=2, n_clusters=32,
                    neighbors=8, batch=2)
    inp = {k: v.to(dev) for k, v in wl.make_inputs(cfg).items()}
    kw = dict(window=cfg.window, budget=cfg.budget, pool_kernel=cfg.pool_kernel, topk_nodes=cfg.topk_nodes,
              neighbors=cfg.neighbors, rounds=cfg.rounds, decay=cfg.decay)
    p = gk.make_params(inp["K"], Qw=inp["Qw"], V=inp["V"], **kw)
    clean = gk.alloc_workspace(p, dev)
    want = gk.alloc_outputs(p, inp["K"])
    gk.graphkv_compress(p, inp["Qw"], inp["K"], inp["V"], want[0], want[1], want[2], want[3], clean)
    assert gk.graphkv_read_status(clean) == gk.OK
    g = torch.Generator(device="cpu").manual_seed(7)
    if two_kernels:
        os.environ["GRAPHKV_TWO_SCORE_KERNELS"] = "1"
    try:
        for fill in (0xFF, None):
            dirty = torch.empty_like(clean)                       # uint8
            if fill is None:
                dirty.copy_(torch.randint(0, 256, (clean.numel(),), dtype=torch.uint8, generator=g))
            else:
                dirty.fill_(fill)
            got = gk.alloc_outputs(p, inp["K"])
            for _ in range(2):
                gk.graphkv_compress(p, inp["Qw"], inp["K"], inp["V"], got[0], got[1], got[2], got[3], dirty)
                assert gk.graphkv_read_status(dirty) == gk.OK
                for a, b in zip(got, want):
                    assert torch.equal(a.view(torch.uint8), b.view(torch.uint8))
    finally:
        os.environ.pop("GRAPHKV_TWO_SCORE_KERNELS", None)
