"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, and rejects bad arguments before touching the device."""
import ctypes as C
import os
import re

import pytest
import torch

from paper_2509_00388_b200 import binding as gk
from paper_2509_00388_b200 import build as gk_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    gk_build.build()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "graphkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(graphkv_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert set(names) >= {"graphkv_score", "graphkv_propagate", "graphkv_select_gather",
                          "graphkv_compress", "graphkv_workspace_bytes"}
    lib = C.CDLL(gk.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in graphkv.h but not exported"
    assert set(gk.EXPORTS) == set(names)


def test_params_struct_matches_header_size():
    # 14 four-byte fields + 9 int64 strides + 2 four-byte fields
    assert C.sizeof(gk.Params) == 14 * 4 + 9 * 8 + 2 * 4


def _params(**kw):
    K = torch.empty(1, 2, 104, 128, dtype=torch.bfloat16)
    Q = torch.empty(1, 4, 4, 128, dtype=torch.bfloat16)
    base = dict(window=4, budget=10, pool_kernel=7, topk_nodes=3, neighbors=2, rounds=1, decay=1.0)
    base.update(kw)
    return gk.make_params(K, Qw=Q, V=K, **base)


def test_workspace_bytes_positive_and_monotone():
    a = gk.workspace_bytes(_params())
    b = gk.workspace_bytes(_params(topk_nodes=30))
    assert a > 0 and b > a and a % 256 == 0


@pytest.mark.parametrize("bad", [
    dict(budget=0), dict(budget=101), dict(pool_kernel=4), dict(pool_kernel=0),
    dict(topk_nodes=-1), dict(topk_nodes=101), dict(neighbors=100), dict(rounds=-1),
    dict(decay=1.5), dict(decay=-0.1), dict(decay=float("nan")),
])
def test_invalid_params_are_rejected_on_the_host(bad):
    p = _params(**bad)
    assert gk.workspace_bytes(p) == 0
    rc = gk.lib().graphkv_compress(C.byref(p), 16, 16, 16, 16, 16, 16, None, 256, 1 << 30, None)
    assert rc == gk.ERR_INVALID_ARG


def test_unsupported_shapes():
    p = _params()
    p.head_dim = 96                                       # 128 and 64 are served
    assert gk.lib().graphkv_score(C.byref(p), 16, 16, 16, 256, 1 << 30, None) == gk.ERR_UNSUPPORTED
    p = _params()
    p.n_q_heads, p.window, p.seq_len = 64, 64, 164      # G*W = 2048 rows
    assert gk.lib().graphkv_score(C.byref(p), 16, 16, 16, 256, 1 << 30, None) == gk.ERR_UNSUPPORTED
    p = _params()
    p.n_q_heads = 5                                       # not a multiple of the KV heads
    assert gk.lib().graphkv_score(C.byref(p), 16, 16, 16, 256, 1 << 30, None) == gk.ERR_INVALID_ARG


def test_null_pointers_misalignment_and_workspace():
    p = _params()
    need = gk.workspace_bytes(p)
    L = gk.lib()
    assert L.graphkv_score(C.byref(p), None, 16, 16, 256, need, None) == gk.ERR_INVALID_ARG
    assert L.graphkv_score(C.byref(p), 16, 24, 16, 256, need, None) == gk.ERR_INVALID_ARG
    assert L.graphkv_score(C.byref(p), 16, 16, 16, None, need, None) == gk.ERR_WORKSPACE
    assert L.graphkv_score(C.byref(p), 16, 16, 16, 256, need - 1, None) == gk.ERR_WORKSPACE
    assert L.graphkv_score(C.byref(p), 16, 16, 16, 128, need, None) == gk.ERR_WORKSPACE
    assert L.graphkv_select_gather(C.byref(p), 16, 16, None, None, None, 16, 256, need,
                                   None) == gk.ERR_INVALID_ARG       # K without K_out
    p.k_stride[2] = 100                                                 # rows would overlap
    assert L.graphkv_score(C.byref(p), 16, 16, 16, 256, need, None) == gk.ERR_INVALID_ARG


def test_status_strings_and_neighbour_rule():
    assert gk.status_string(gk.OK) == "ok"
    assert "workspace" in gk.status_string(gk.ERR_WORKSPACE)
    assert [gk.resolve_neighbors(n, 0) for n in (512, 16384, 32768, 131072)] == [1, 16, 32, 32]
    assert gk.resolve_neighbors(5, 0) == 1 and gk.resolve_neighbors(1, 0) == 0
    assert gk.resolve_neighbors(32768, 7) == 7


def test_binding_has_no_cpu_route():
    import inspect
    src = inspect.getsource(gk)
    assert "oracle" not in src


def test_variant_fields_and_entry_points_validate_on_the_host():
    lib = gk.lib()
    for bad in (dict(signal=3), dict(signal=-1), dict(reselect=2), dict(pool_mode=2)):
        assert gk.workspace_bytes(_params(**bad)) == 0
    for ok in (dict(signal=gk.SIGNAL_EVICT), dict(reselect=1), dict(pool_mode=gk.POOL_AVG)):
        assert gk.workspace_bytes(_params(**ok)) > 0
    p = _params()
    # edge operands: unknown tensor kind, missing tensor
    assert lib.graphkv_propagate_edges(C.byref(p), 256, None, 0, 7, 256, None, 256, 1 << 30, None) == gk.ERR_INVALID_ARG
    assert lib.graphkv_propagate_edges(C.byref(p), 256, None, gk.TENSOR_V, gk.TENSOR_V, 256, None, 256, 1 << 30,
                                       None) == gk.ERR_INVALID_ARG
    assert lib.graphkv_score_knorm(C.byref(p), None, 256, None) == gk.ERR_INVALID_ARG
    # per-layer budgets: each within 1 .. params.budget, at most 64 layers
    arr = (C.c_int32 * 1)(11)
    assert lib.graphkv_compress_layers(C.byref(p), arr, 256, 256, 256, 256, 256, 256, None, 256, 1 << 30,
                                       None) == gk.ERR_INVALID_ARG
    assert lib.graphkv_compress_layers(C.byref(p), None, 256, 256, 256, 256, 256, 256, None, 256, 1 << 30,
                                       None) == gk.ERR_INVALID_ARG
    # decode attention: shape checks and workspace sizing without a device
    q = torch.empty(1, 4, 128, dtype=torch.bfloat16)
    K = torch.empty(1, 2, 100, 128, dtype=torch.bfloat16)
    dp = gk.decode_params(q, K, K)
    need = int(lib.graphkv_decode_workspace_bytes(C.byref(dp)))
    assert need > 0 and need % 256 == 0
    assert lib.graphkv_decode_attention(C.byref(dp), 256, 256, 256, 256, 256, need - 1, None) == gk.ERR_WORKSPACE
    q9 = torch.empty(1, 18, 128, dtype=torch.bfloat16)       # 9 query heads per KV head: beyond the kernel
    assert int(lib.graphkv_decode_workspace_bytes(C.byref(gk.decode_params(q9, K, K)))) == 0
