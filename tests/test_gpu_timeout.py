"""The bounded device-side waits: a wait that runs out must end the kernel by itself, leave
GRAPHKV_ERR_TIMEOUT in the status word and leave the workspace usable.

The wait is made to run out on the host side only: the limit is shortened through
GRAPHKV_WAIT_CYCLES and a test hook makes the MMA issuer of the statistics sweep leave out one
arrival (the one that announces its first accumulator), so the epilogue's wait for it, the
issuer's wait for the buffer to come back and the producer's wait for a free stage all reach
their limit and drain.  A second hook makes every CTA of the kernel that runs both sweeps leave
out its announcement at the hand-over between the passes, so the wait for the unit's other chunks
runs out.  Nothing faults, traps or waits without a limit."""
import os

import pytest
import torch

from paper_2509_00388_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("hook,two_kernels", [("1", False), ("1", True), ("2", False)])
def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_exact(hook, two_kernels):
    from paper_2509_00388_b200 import binding as gk
    gk.lib()
    dev = torch.device("cuda:0")
    cfg = wl.scaled(wl.LLAMA_32K, n_prefix=3000, budget=64, n_q_heads=8, n_kv_heads=2, n_clusters=16)
    inp = wl.make_inputs(cfg)
    Qd, Kd = inp["Qw"].to(dev), inp["K"].to(dev)
    p = gk.make_params(Kd, Qw=Qd, window=cfg.window, pool_kernel=cfg.pool_kernel)
    ws = gk.alloc_workspace(p, dev)
    want = torch.empty((p.batch, p.n_kv_heads, cfg.n_prefix), dtype=torch.float32, device=dev)
    gk.graphkv_score(p, Qd, Kd, want, ws)
    assert gk.graphkv_read_status(ws) == gk.OK

    got = torch.empty_like(want)
    os.environ["GRAPHKV_WAIT_CYCLES"] = "2000000"           # about a millisecond
    os.environ["GRAPHKV_DEBUG_WITHHOLD_COMMIT"] = hook
    if two_kernels:
        os.environ["GRAPHKV_TWO_SCORE_KERNELS"] = "1"
    try:
        gk.graphkv_score(p, Qd, Kd, got, ws)
        status = gk.graphkv_read_status(ws)                 # synchronises: the kernels returned
    finally:
        os.environ.pop("GRAPHKV_WAIT_CYCLES", None)
        os.environ.pop("GRAPHKV_DEBUG_WITHHOLD_COMMIT", None)
        os.environ.pop("GRAPHKV_TWO_SCORE_KERNELS", None)
    assert status == gk.ERR_TIMEOUT
    assert "timed out" in gk.status_string(status)

    # the same workspace, a normal call: the status is clean again and the scores are bit-exact
    gk.graphkv_score(p, Qd, Kd, got, ws)
    assert gk.graphkv_read_status(ws) == gk.OK
    assert torch.equal(got, want)
