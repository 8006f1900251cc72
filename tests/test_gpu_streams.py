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
