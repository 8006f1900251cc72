"""graphkv_score_noalloc: the scoring call for callers that may not allocate device memory (code
running inside a region a framework has closed to cudaMalloc, or in a process whose memory was
handed out in full at start-up).  Its scratch is an array inside the library image, so these
tests check that it gives what graphkv_score gives with a caller-made workspace, twice in a row
(the array keeps the previous call's contents), and that it refuses problems that do not fit.

Collected last on purpose: a run that stops at the first failure has then run everything else.
"""
import pytest
import torch

from paper_2509_00388_b200 import binding as gk
from paper_2509_00388_b200 import build as gk_build
from paper_2509_00388_b200 import workloads as wl
from tests import parity_util as pu


@pytest.fixture(scope="module", autouse=True)
def built():
    gk_build.build()


def _case(**kw):
    base = dict(n_prefix=6000, budget=64, n_q_heads=8, n_kv_heads=2, n_clusters=32)
    base.update(kw)
    return wl.scaled(wl.LLAMA_32K, **base)


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_noalloc_score_matches_the_workspace_call_twice_in_a_row(dtype):
    gk.lib()
    dev = torch.device("cuda:0")
    for seed, n in ((0, 6000), (1, 4321)):          # two calls in a row, different sizes
        cfg = _case(dtype=dtype, n_prefix=n, seed=seed)
        inp = wl.make_inputs(cfg)
        Qd, Kd = inp["Qw"].to(dev), inp["K"].to(dev)
        p = gk.make_params(Kd, Qw=Qd, window=cfg.window, pool_kernel=cfg.pool_kernel)
        assert 0 < gk.builtin_scratch_needed(p) <= gk.BUILTIN_SCRATCH_BYTES
        want = torch.empty((p.batch, p.n_kv_heads, n), dtype=torch.float32, device=dev)
        ws = gk.alloc_workspace(p, dev)
        gk.graphkv_score(p, Qd, Kd, want, ws)
        assert gk.graphkv_read_status(ws) == gk.OK
        got = torch.full_like(want, float("nan"))
        torch.cuda.synchronize(dev)
        # free bytes as the driver counts them: an allocation made behind torch's back shows here
        free_before = torch.cuda.mem_get_info(dev)[0]
        before = torch.cuda.memory_allocated(dev)
        gk.graphkv_score_noalloc(p, Qd, Kd, got)
        assert gk.graphkv_read_status_noalloc(dev) == gk.OK
        assert torch.cuda.memory_allocated(dev) == before
        if seed > 0:        # the very first call may load the kernels' module; later ones may not grow
            assert torch.cuda.mem_get_info(dev)[0] >= free_before
        assert pu.score_rel_err(got.cpu(), want.cpu()) <= pu.SCORE_RTOL
        assert torch.equal(got, want)               # same kernels, same arithmetic


def test_noalloc_score_refuses_what_does_not_fit():
    # host-side check only: nothing is launched, so no GPU is needed
    K = torch.empty(8, 8, 131072 + 32, 128, dtype=torch.bfloat16, device="meta")
    Q = torch.empty(8, 32, 32, 128, dtype=torch.bfloat16, device="meta")
    p = gk.make_params(K, Qw=Q, window=32, pool_kernel=7)
    assert gk.builtin_scratch_needed(p) > gk.BUILTIN_SCRATCH_BYTES
    code = gk.lib().graphkv_score_noalloc(__import__("ctypes").byref(p), 256, 256, 256, None)
    assert code == gk.ERR_BUILTIN_SCRATCH
    assert "built-in" in gk.status_string(code)
