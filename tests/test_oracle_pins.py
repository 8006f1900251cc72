"""Pins of the CPU oracle against things other than itself: numpy brute force of the plain
definitions (softmax attention, normalised matmul, argsort), closed forms, invariants and the
special cases named in the paper (T = 0 is the base method; Eq. 5's product over a fixed graph).
"""
import math

import numpy as np
import pytest
import torch
from hypothesis import given, settings, strategies as st

from oracle import graphkv_oracle as okv

# ----------------------------------------------------------------------------- helpers


def rand_unit(seed, G=2, W=4, D=16, N=40, scale=1.0):
    rng = np.random.default_rng(seed)
    Qg = torch.from_numpy(rng.standard_normal((G, W, D)).astype(np.float32) * scale)
    Kh = torch.from_numpy(rng.standard_normal((N + W, D)).astype(np.float32))
    return Qg, Kh


def brute_attention_mass(Qg, Kh):
    """Library definition: softmax(Q K^T / sqrt(D)) with a causal mask on the window block,
    summed over all G*W rows; returns the [L] column mass in fp64."""
    G, W, D = Qg.shape
    L = Kh.shape[0]
    N = L - W
    Q = Qg.double().numpy().reshape(G * W, D)
    K = Kh.double().numpy()
    logits = Q @ K.T / math.sqrt(D)
    r = np.tile(np.arange(W), G)[:, None]
    j = np.arange(L)[None, :]
    logits = np.where(j <= N + r, logits, -np.inf)
    logits -= logits.max(axis=1, keepdims=True)
    P = np.exp(logits)
    P /= P.sum(axis=1, keepdims=True)
    return P.sum(axis=0)


def brute_maxpool(a, kp):
    half = (kp - 1) // 2
    padded = np.concatenate([np.full(half, -np.inf), a, np.full(half, -np.inf)])
    win = np.lib.stride_tricks.sliding_window_view(padded, kp)
    return win.max(axis=1)


def brute_topk(x, k, skip=-1):
    """(value desc, index asc) via a stable lexsort on the fp32 values."""
    x = np.asarray(x, dtype=np.float32)
    idx = np.arange(x.shape[0])
    keep = idx != skip
    order = np.lexsort((idx[keep], -x[keep].astype(np.float64)))
    return idx[keep][order][:k]


def brute_cosine(Kh, N):
    K = Kh.double().numpy()[:N]
    Kn = K / np.maximum(np.linalg.norm(K, axis=1, keepdims=True), 1e-12)
    return Kn @ Kn.T


# ----------------------------------------------------------------------------- step (I)


@pytest.mark.parametrize("seed,G,W,D,N", [(0, 1, 4, 16, 40), (1, 2, 4, 16, 33), (2, 4, 8, 32, 100),
                                          (3, 3, 1, 8, 5), (4, 2, 6, 128, 64)])
def test_score_matches_bruteforce_softmax_attention(seed, G, W, D, N):
    Qg, Kh = rand_unit(seed, G, W, D, N, scale=2.0)
    a, s = okv.score_unit(Qg, Kh, pool_kernel=1)
    ref = brute_attention_mass(Qg, Kh)
    np.testing.assert_allclose(a.numpy(), ref[:N], rtol=1e-12, atol=1e-15)
    # kp = 1 is the identity, and the fp32 output is the rounded fp64 mass
    np.testing.assert_array_equal(s.numpy(), ref[:N].astype(np.float32))


def test_score_total_mass_is_rows_minus_window_mass():
    Qg, Kh = rand_unit(7, G=2, W=5, D=16, N=50, scale=3.0)
    a, _ = okv.score_unit(Qg, Kh, pool_kernel=1)
    ref = brute_attention_mass(Qg, Kh)
    G, W, _ = Qg.shape
    assert abs(ref.sum() - G * W) < 1e-9
    assert abs(a.sum().item() + ref[50:].sum() - G * W) < 1e-9


def test_score_zero_queries_closed_form():
    # all logits 0: row r spreads 1/(N+r+1) over its visible keys
    G, W, D, N = 3, 6, 8, 29
    Qg = torch.zeros(G, W, D)
    _, Kh = rand_unit(5, G, W, D, N)
    a, s = okv.score_unit(Qg, Kh, pool_kernel=7)
    expect = G * sum(1.0 / (N + r + 1) for r in range(W))
    np.testing.assert_allclose(a.numpy(), np.full(N, expect), rtol=1e-13)
    np.testing.assert_array_equal(s.numpy(), np.full(N, np.float32(expect)))


def test_score_causal_mask_in_window_block():
    # a window key that only later rows may see must not receive mass from earlier rows:
    # with W = 2 and a huge last window key, row 0 must ignore it.
    D, N, W = 4, 3, 2
    Kh = torch.zeros(N + W, D)
    Kh[N + 1, 0] = 50.0                      # visible to row 1 only
    Qg = torch.zeros(1, W, D)
    Qg[0, :, 0] = 1.0
    a, _ = okv.score_unit(Qg, Kh, pool_kernel=1)
    row0 = 1.0 / (N + 1)                      # uniform over keys 0..N
    z1 = N + 1 + math.exp(50.0 / math.sqrt(D))
    expect = row0 + 1.0 / z1
    np.testing.assert_allclose(a.numpy(), np.full(N, expect), rtol=1e-12)


def test_score_scale_is_inverse_sqrt_d_and_operands_not_transposed():
    # single query, two keys: mass ratio must be exp((q.k0 - q.k1)/sqrt(D))
    D = 9
    q = torch.arange(1, D + 1, dtype=torch.float32).reshape(1, 1, D) / 3
    k0 = torch.linspace(-1, 1, D)
    k1 = torch.linspace(1, -0.5, D)
    kw = torch.zeros(D)
    Kh = torch.stack([k0, k1, kw])
    a, _ = okv.score_unit(q, Kh, pool_kernel=1)
    qv = q.reshape(D).double()
    ratio = math.exp(((qv @ k0.double()) - (qv @ k1.double())).item() / math.sqrt(D))
    assert abs(a[0].item() / a[1].item() - ratio) < 1e-12 * ratio


@pytest.mark.parametrize("kp", [1, 3, 7, 9])
def test_pooling_matches_sliding_window_max(kp):
    Qg, Kh = rand_unit(11, G=2, W=4, D=16, N=37, scale=4.0)
    a, s = okv.score_unit(Qg, Kh, pool_kernel=kp)
    np.testing.assert_array_equal(s.numpy(), brute_maxpool(a.numpy(), kp).astype(np.float32))
    assert np.all(s.numpy() >= a.numpy().astype(np.float32))


@pytest.mark.parametrize("jstar", [0, 1, 17, 35, 36])
def test_pooling_spike_gives_clipped_plateau(jstar):
    G, W, D, N, kp = 1, 2, 8, 37, 7
    Kh = torch.zeros(N + W, D)
    Kh[jstar, 0] = 30.0
    Qg = torch.zeros(G, W, D)
    Qg[:, :, 0] = 3.0
    a, s = okv.score_unit(Qg, Kh, pool_kernel=kp)
    lo, hi = max(0, jstar - 3), min(N - 1, jstar + 3)
    plateau = np.zeros(N, dtype=bool)
    plateau[lo:hi + 1] = True
    top = np.float32(a[jstar].item())
    assert np.all(s.numpy()[plateau] == top)
    assert np.all(s.numpy()[~plateau] < top)


# ----------------------------------------------------------------------------- top-k rule


@given(st.integers(0, 10_000), st.integers(1, 60), st.integers(1, 4))
@settings(max_examples=60, deadline=None)
def test_topk_matches_lexsort_with_ties(seed, n, levels):
    rng = np.random.default_rng(seed)
    x = rng.integers(0, levels + 1, size=n).astype(np.float32)   # many exact ties
    k = int(rng.integers(1, n + 1))
    got = okv.topk(torch.from_numpy(x), k).numpy()
    np.testing.assert_array_equal(got, brute_topk(x, k))


def test_topk_skip_excludes_index():
    x = torch.tensor([5.0, 9.0, 9.0, 1.0, 7.0])
    assert okv.topk(x, 2, skip=1).tolist() == [2, 4]
    assert okv.topk(x, 3).tolist() == [1, 2, 4]


def test_constant_scores_keep_lowest_indices():
    # zero queries => constant scores => every selection takes the lowest indices
    G, W, D, N, B = 2, 4, 8, 50, 9
    rng = np.random.default_rng(3)
    K = torch.from_numpy(rng.standard_normal((1, 1, N + W, D)).astype(np.float32))
    V = torch.from_numpy(rng.standard_normal((1, 1, N + W, D)).astype(np.float32))
    Qw = torch.zeros(1, G, W, D)
    K_out, V_out, idx, _ = okv.compress(Qw, K, V, window=W, budget=B, pool_kernel=7,
                                        topk_nodes=0, neighbors=0, rounds=0, decay=1.0)
    assert idx[0, 0].tolist() == list(range(B))
    assert torch.equal(K_out[0, 0], torch.cat([K[0, 0, :B], K[0, 0, N:]]))
    assert torch.equal(V_out[0, 0], torch.cat([V[0, 0, :B], V[0, 0, N:]]))


# ----------------------------------------------------------------------------- Eq. 1 edges


@pytest.mark.parametrize("seed", [0, 1])
def test_edges_match_normalised_matmul(seed):
    _, Kh = rand_unit(seed, G=1, W=3, D=24, N=31)
    cos = brute_cosine(Kh, 31)
    for i in (0, 7, 30):
        e = okv.edges_unit(Kh, 31, i).numpy()
        np.testing.assert_allclose(e, cos[i], rtol=1e-12, atol=1e-14)


def test_edges_invariant_under_positive_row_rescaling():
    _, Kh = rand_unit(2, G=1, W=3, D=24, N=31)
    scale = torch.from_numpy(np.random.default_rng(0).uniform(0.1, 9.0, size=(34, 1))).float()
    e0 = okv.edges_unit(Kh, 31, 5).numpy()
    e1 = okv.edges_unit(Kh * scale, 31, 5).numpy()
    np.testing.assert_allclose(e0, e1, rtol=1e-6, atol=1e-7)  # fp32 rescale rounds the inputs


def test_edges_zero_norm_key_gives_zero():
    _, Kh = rand_unit(2, G=1, W=3, D=8, N=10)
    Kh[4] = 0.0
    e = okv.edges_unit(Kh, 10, 2).numpy()
    assert e[4] == 0.0
    assert okv.edges_unit(Kh, 10, 4).abs().max().item() == 0.0


# ----------------------------------------------------------------------------- Eq. 2-5


def _prop(Kh, s, N, **kw):
    args = dict(topk_nodes=3, neighbors=4, rounds=1, decay=1.0)
    args.update(kw)
    return okv.propagate_unit(Kh, s, N, **args)


def test_sources_are_topk_by_score_and_neighbours_topm_by_cosine():
    N = 45
    _, Kh = rand_unit(4, G=1, W=3, D=16, N=N)
    s = torch.from_numpy(np.random.default_rng(1).random(N).astype(np.float32))
    _, src, nbr, nbr_e = _prop(Kh, s, N, topk_nodes=5, neighbors=6)
    np.testing.assert_array_equal(src.numpy(), brute_topk(s.numpy(), 5))
    cos = brute_cosine(Kh, N)
    for a, i in enumerate(src.tolist()):
        want = brute_topk(cos[i].astype(np.float32), 6, skip=i)
        np.testing.assert_array_equal(nbr[a].numpy(), want)
        assert i not in nbr[a].tolist()
        np.testing.assert_allclose(nbr_e[a].numpy(), cos[i][want], rtol=1e-12)


@pytest.mark.parametrize("T,lam", [(1, 1.0), (2, 0.5), (3, 0.25), (4, 1.0)])
def test_rounds_closed_form_product_over_fixed_graph(T, lam):
    N = 60
    _, Kh = rand_unit(8, G=1, W=3, D=16, N=N)
    s = torch.from_numpy(np.random.default_rng(2).random(N).astype(np.float32) + 0.1)
    out, src, nbr, nbr_e = _prop(Kh, s, N, topk_nodes=6, neighbors=7, rounds=T, decay=lam)
    cos = brute_cosine(Kh, N)
    f = np.ones(N)
    for a, i in enumerate(brute_topk(s.numpy(), 6)):
        for j in brute_topk(cos[i].astype(np.float32), 7, skip=i):
            f[j] *= 1.0 - lam * max(cos[i, j], 0.0)
    expect = (s.double().numpy() * f ** T).astype(np.float32)
    np.testing.assert_allclose(out.numpy(), expect, rtol=3e-7)
    changed = np.flatnonzero(out.numpy() != s.numpy())
    assert changed.size <= 6 * 7
    assert np.all(out.numpy() <= s.numpy())          # scores never increase
    assert set(changed.tolist()) <= set(nbr.numpy().reshape(-1).tolist())


def test_zero_rounds_and_zero_decay_are_identities():
    N = 30
    _, Kh = rand_unit(9, G=1, W=3, D=16, N=N)
    s = torch.from_numpy(np.random.default_rng(3).random(N).astype(np.float32))
    out0, *_ = _prop(Kh, s, N, rounds=0)
    out1, *_ = _prop(Kh, s, N, rounds=3, decay=0.0)
    assert torch.equal(out0, s) and torch.equal(out1, s)


def test_single_source_full_neighbourhood_is_dense_cosine_row():
    N = 25
    _, Kh = rand_unit(10, G=1, W=3, D=16, N=N)
    s = torch.ones(N)
    s[11] = 2.0
    lam = 0.7
    out, src, _, _ = _prop(Kh, s, N, topk_nodes=1, neighbors=N - 1, rounds=1, decay=lam)
    assert src.tolist() == [11]
    cos = brute_cosine(Kh, N)[11]
    expect = s.double().numpy() * (1.0 - lam * np.maximum(cos, 0.0))
    expect[11] = 2.0                                  # j = i is excluded by Eq. 3
    np.testing.assert_allclose(out.numpy(), expect.astype(np.float32), rtol=2e-7)


def test_exact_duplicate_of_source_is_zeroed_and_orthogonal_keys_untouched():
    D, N = 8, 8
    Kh = torch.zeros(N + 2, D)
    for j in range(N):
        Kh[j, j % D] = 1.0 + j                        # mutually orthogonal axes, varied norms
    Kh[5] = 3.0 * Kh[2]                                # same direction as key 2
    s = torch.tensor([1, 1, 9, 1, 1, 4, 1, 1], dtype=torch.float32)
    out, src, nbr, _ = _prop(Kh, s, N, topk_nodes=1, neighbors=3, rounds=1, decay=1.0)
    assert src.tolist() == [2]
    assert nbr[0].tolist()[0] == 5                     # cosine 1 ranks first
    expect = s.clone()
    expect[5] = 0.0
    assert torch.equal(out, expect)                    # e = 0 neighbours keep their score


def test_negative_cosine_is_clamped():
    D, N = 4, 3
    Kh = torch.zeros(N + 1, D)
    Kh[0, 0] = 1.0
    Kh[1, 0] = -1.0
    Kh[2, 0] = -2.0
    s = torch.tensor([5.0, 1.0, 1.0])
    out, *_ = _prop(Kh, s, N, topk_nodes=1, neighbors=2, rounds=2, decay=1.0)
    assert torch.equal(out, s)


def test_overlapping_neighbourhoods_multiply():
    # two sources pointing the same way share neighbour 2: its factor is the product (Eq. 5)
    D, N = 4, 4
    Kh = torch.zeros(N + 1, D)
    Kh[0] = torch.tensor([1.0, 0.0, 0, 0])
    Kh[1] = torch.tensor([1.0, 1.0, 0, 0])
    Kh[2] = torch.tensor([1.0, 0.5, 0, 0])
    Kh[3] = torch.tensor([0.0, 0.0, 1, 0])
    s = torch.tensor([9.0, 8.0, 1.0, 1.0])
    lam = 0.5
    out, src, nbr, _ = _prop(Kh, s, N, topk_nodes=2, neighbors=1, rounds=1, decay=lam)
    assert src.tolist() == [0, 1] and nbr.reshape(-1).tolist() == [2, 2]
    cos = brute_cosine(Kh, N)
    expect = 1.0 * (1 - lam * cos[0, 2]) * (1 - lam * cos[1, 2])
    assert abs(out[2].item() - expect) < 1e-6
    assert out[0].item() == 9.0 and out[1].item() == 8.0 and out[3].item() == 1.0


def test_adaptive_neighbour_rule():
    assert okv.resolve_neighbors(512, 0) == 1
    assert okv.resolve_neighbors(16384, 0) == 16
    assert okv.resolve_neighbors(32768, 0) == 32
    assert okv.resolve_neighbors(131072, 0) == 32
    assert okv.resolve_neighbors(32768, 5) == 5
    # the length rule is a factor of 1e-3 (not 2^-10), floored
    assert okv.resolve_neighbors(5000, 0) == 5
    assert okv.resolve_neighbors(31999, 0) == 31
    assert okv.resolve_neighbors(1999, 0) == 1 and okv.resolve_neighbors(2000, 0) == 2


# ----------------------------------------------------------------------------- step (IV)


@given(st.integers(0, 10_000), st.integers(2, 80))
@settings(max_examples=40, deadline=None)
def test_select_gather_matches_argsort(seed, n):
    rng = np.random.default_rng(seed)
    W, D = 3, 4
    B = int(rng.integers(1, n + 1))
    s = rng.integers(0, 6, size=(1, 1, n)).astype(np.float32)     # ties on purpose
    K = torch.from_numpy(rng.standard_normal((1, 1, n + W, D)).astype(np.float32))
    V = torch.from_numpy(rng.standard_normal((1, 1, n + W, D)).astype(np.float32))
    K_out, V_out, idx = okv.select_gather(torch.from_numpy(s), K, V, window=W, budget=B)
    want = np.sort(brute_topk(s[0, 0], B))
    np.testing.assert_array_equal(idx[0, 0].numpy(), want)
    assert len(set(want.tolist())) == B
    assert torch.equal(K_out[0, 0, :B], K[0, 0, want]) and torch.equal(K_out[0, 0, B:], K[0, 0, n:])
    assert torch.equal(V_out[0, 0, :B], V[0, 0, want]) and torch.equal(V_out[0, 0, B:], V[0, 0, n:])


def test_gather_is_bit_exact_for_bf16():
    rng = np.random.default_rng(0)
    n, W, D, B = 40, 4, 8, 10
    K = torch.from_numpy(rng.standard_normal((2, 2, n + W, D)).astype(np.float32)).bfloat16()
    V = torch.from_numpy(rng.standard_normal((2, 2, n + W, D)).astype(np.float32)).bfloat16()
    s = torch.from_numpy(rng.random((2, 2, n)).astype(np.float32))
    K_out, V_out, idx = okv.select_gather(s, K, V, window=W, budget=B)
    for b in range(2):
        for h in range(2):
            ii = idx[b, h].long()
            assert torch.equal(K_out[b, h].view(torch.int16),
                               torch.cat([K[b, h, ii], K[b, h, n:]]).view(torch.int16))
            assert torch.equal(V_out[b, h].view(torch.int16),
                               torch.cat([V[b, h, ii], V[b, h, n:]]).view(torch.int16))


# ----------------------------------------------------------------------------- whole path


def _tiny_inputs(seed=0, b=2, hq=4, hkv=2, N=96, W=4, D=16):
    rng = np.random.default_rng(seed)
    Qw = torch.from_numpy(rng.standard_normal((b, hq, W, D)).astype(np.float32) * 2)
    K = torch.from_numpy(rng.standard_normal((b, hkv, N + W, D)).astype(np.float32))
    V = torch.from_numpy(rng.standard_normal((b, hkv, N + W, D)).astype(np.float32))
    return Qw, K, V


def test_zero_rounds_reproduces_plain_window_attention_topb():
    Qw, K, V = _tiny_inputs()
    W, B = 4, 12
    _, _, idx, s = okv.compress(Qw, K, V, window=W, budget=B, pool_kernel=7, topk_nodes=5,
                                neighbors=3, rounds=0, decay=1.0)
    s0 = okv.score(Qw, K, W, 7)
    assert torch.equal(s, s0)
    for b in range(2):
        for h in range(2):
            want = np.sort(brute_topk(s0[b, h].numpy(), B))
            np.testing.assert_array_equal(idx[b, h].numpy(), want)


def test_compress_is_the_composition_of_its_stages_and_heads_map_to_their_group():
    Qw, K, V = _tiny_inputs(seed=1)
    W, B = 4, 10
    kw = dict(window=W, budget=B, pool_kernel=3, topk_nodes=4, neighbors=3, rounds=2, decay=0.5)
    K_out, V_out, idx, s = okv.compress(Qw, K, V, **kw)
    s0 = okv.score(Qw, K, W, 3)
    # GQA grouping: KV head h takes query heads [h*G, (h+1)*G)
    for b in range(2):
        for h in range(2):
            _, su = okv.score_unit(Qw[b, 2 * h:2 * h + 2], K[b, h], 3)
            assert torch.equal(su, s0[b, h])
    s1, src = okv.propagate(K, s0, W, 4, 3, 2, 0.5)
    assert torch.equal(s1, s)
    assert np.all(s1.numpy() <= s0.numpy())
    K2, V2, idx2 = okv.select_gather(s1, K, V, W, B)
    assert torch.equal(idx, idx2) and torch.equal(K_out, K2) and torch.equal(V_out, V2)
    # counts: exactly B distinct ascending prefix positions, window rows retained
    N = K.shape[2] - W
    for b in range(2):
        for h in range(2):
            ii = idx[b, h].numpy()
            assert np.all(np.diff(ii) > 0) and ii.min() >= 0 and ii.max() < N
            assert torch.equal(K_out[b, h, B:], K[b, h, N:])
            np.testing.assert_array_equal(src[b, h].numpy(), brute_topk(s0[b, h].numpy(), 4))


def test_permuting_prefix_tokens_permutes_the_kept_set_without_pooling():
    Qw, K, V = _tiny_inputs(seed=2, b=1, hq=2, hkv=1, N=64)
    W, B, N = 4, 9, 64
    kw = dict(window=W, budget=B, pool_kernel=1, topk_nodes=3, neighbors=4, rounds=1, decay=1.0)
    _, _, idx, _ = okv.compress(Qw, K, V, **kw)
    perm = torch.from_numpy(np.random.default_rng(5).permutation(N))
    full = torch.cat([perm, torch.arange(N, N + W)])
    _, _, idx_p, _ = okv.compress(Qw, K[:, :, full], V[:, :, full], **kw)
    # position t of the permuted input holds original token perm[t]
    assert sorted(perm[idx_p[0, 0].long()].tolist()) == idx[0, 0].tolist()


def test_decay_changes_selection_away_from_duplicates():
    # the method's purpose: with duplicates of a top token, propagation drops the copies
    D, N, W = 8, 12, 1
    rng = np.random.default_rng(0)
    Kp = rng.standard_normal((N, D)).astype(np.float32)
    Kp[3] = Kp[2]
    Kp[4] = Kp[2]                                        # tokens 2,3,4 identical
    q = (4.0 * Kp[2]).reshape(1, 1, 1, D)
    K = torch.from_numpy(np.concatenate([Kp, np.zeros((W, D), np.float32)])).reshape(1, 1, N + W, D)
    V = K.clone()
    base = dict(window=W, budget=3, pool_kernel=1, topk_nodes=1, neighbors=2, decay=1.0)
    _, _, idx0, _ = okv.compress(torch.from_numpy(q), K, V, rounds=0, **base)
    _, _, idx1, s1 = okv.compress(torch.from_numpy(q), K, V, rounds=1, **base)
    assert idx0[0, 0].tolist() == [2, 3, 4]
    assert 2 in idx1[0, 0].tolist() and 3 not in idx1[0, 0].tolist() and 4 not in idx1[0, 0].tolist()
    assert s1[0, 0, 3].item() == 0.0 and s1[0, 0, 4].item() == 0.0


# ----------------------------------------------------------------------------- KNorm initial score


def test_knorm_score_is_the_reciprocal_key_norm_of_the_prefix():
    rng = np.random.default_rng(3)
    K = torch.from_numpy(rng.standard_normal((2, 2, 37 + 5, 16)).astype(np.float32) * 3)
    K[0, 1, 4] = 0.0                                   # a zero key: norm floored, score finite
    s = okv.score_knorm(K, window=5)
    assert s.shape == (2, 2, 37)
    want = 1.0 / np.maximum(np.linalg.norm(K[:, :, :37].double().numpy(), axis=-1), 1e-12)
    np.testing.assert_allclose(s.double().numpy(), want, rtol=1e-6)
    assert np.isfinite(s.numpy()).all() and (s.numpy() > 0).all()
    # ranks like ascending L2 norm: the key of lowest norm scores highest
    norms = np.linalg.norm(K[1, 0, :37].double().numpy(), axis=-1)
    assert int(s[1, 0].argmax()) == int(norms.argmin())
    # scaling a key by c scales its score by 1/c
    K2 = K.clone()
    K2[1, 1, 7] *= 4.0
    assert abs(okv.score_knorm(K2, 5)[1, 1, 7].item() * 4.0 - s[1, 1, 7].item()) < 1e-6


# ----------------------------------------------------------------------------- variants


def test_average_pooling_matches_the_library_routine():
    # mean over kp positions with zeros outside the row = avg_pool1d with zero padding counted
    for seed, (G, W, D, N, kp) in enumerate([(2, 4, 16, 40, 7), (1, 3, 8, 9, 5), (2, 2, 8, 30, 1)]):
        Qg, Kh = rand_unit(seed, G, W, D, N, scale=2.0)
        a, s = okv.score_unit(Qg, Kh, pool_kernel=kp, pool_mode=okv.POOL_AVG)
        ref = torch.nn.functional.avg_pool1d(a[None, None], kp, stride=1, padding=kp // 2,
                                             count_include_pad=True)[0, 0]
        np.testing.assert_allclose(s.double().numpy(), ref.numpy(), rtol=1e-6)
        assert s.shape[0] == N
    # and through the whole-layer driver
    Qw, K, V = _tiny_inputs(seed=4)
    s_avg = okv.score(Qw, K, 4, 5, pool_mode=okv.POOL_AVG)
    _, su = okv.score_unit(Qw[1, 2:4], K[1, 1], 5, pool_mode=okv.POOL_AVG)
    assert torch.equal(su, s_avg[1, 1])
    assert not torch.equal(s_avg, okv.score(Qw, K, 4, 5))


def brute_propagate(S, A, s, N, k, m, T, lam, signal=0, reselect=False):
    """Eq. 1-5 by definition in numpy fp64: sources = top-k, edges = cosine(S[i], A[j]),
    neighbourhoods = top-m (j != i), T rounds; with reselect the graph is rebuilt every round from
    the scores rounded to fp32."""
    S = S.double().numpy()[:N]
    A = A.double().numpy()[:N]
    Sn = S / np.maximum(np.linalg.norm(S, axis=1, keepdims=True), 1e-12)
    An = A / np.maximum(np.linalg.norm(A, axis=1, keepdims=True), 1e-12)
    cos = np.clip(Sn @ An.T, -1.0, 1.0)
    cur = s.double().numpy().copy()

    def graph(scores32):
        src = brute_topk(scores32, k)
        return src, [brute_topk(cos[i].astype(np.float32), m, skip=i) for i in src]

    src, nbrs = graph(cur.astype(np.float32))
    for t in range(T):
        if reselect and t > 0:
            cur = cur.astype(np.float32).astype(np.float64)
            src, nbrs = graph(cur.astype(np.float32))
        for i, nb in zip(src, nbrs):
            for j in nb:
                e = max(cos[i, j], 0.0)
                if signal == 2:
                    cur[j] = -np.inf
                elif signal == 1:
                    cur[j] *= 1.0 + lam * e
                else:
                    cur[j] *= 1.0 - lam * e
    return cur.astype(np.float32), src


@pytest.mark.parametrize("signal", [0, 1, 2])
@pytest.mark.parametrize("reselect", [0, 1])
def test_signals_and_reselection_match_the_definition(signal, reselect):
    rng = np.random.default_rng(10 * signal + reselect)
    N, W, D = 60, 2, 8
    K = torch.from_numpy(rng.standard_normal((1, 1, N + W, D)).astype(np.float32))
    s0 = torch.from_numpy(rng.random((1, 1, N)).astype(np.float32) + 0.1)
    got, src = okv.propagate(K, s0, W, 4, 3, 3, 0.7, signal=signal, reselect=reselect)
    want, want_src = brute_propagate(K[0, 0], K[0, 0], s0[0, 0], N, 4, 3, 3, 0.7, signal, bool(reselect))
    g, w = got[0, 0].numpy(), want
    assert np.array_equal(np.isinf(g), np.isinf(w))
    np.testing.assert_allclose(g[np.isfinite(g)], w[np.isfinite(w)], rtol=1e-6)
    assert sorted(src[0, 0].tolist()) == sorted(want_src.tolist())
    if signal == 1:
        assert np.all(g >= s0[0, 0].numpy())           # an enhanced signal never lowers a score
    if signal == 2:
        assert np.isinf(g).sum() > 0 and np.all(g[np.isfinite(g)] == s0[0, 0].numpy()[np.isfinite(g)])
    if reselect:
        # re-picking matters: some round takes other sources than the first
        fixed, _ = okv.propagate(K, s0, W, 4, 3, 3, 0.7, signal=signal, reselect=0)
        assert signal == 1 or not torch.equal(fixed, got)


def test_value_and_key_value_edges_match_the_definition():
    rng = np.random.default_rng(7)
    N, W, D = 50, 2, 8
    K = torch.from_numpy(rng.standard_normal((N + W, D)).astype(np.float32))
    V = torch.from_numpy(rng.standard_normal((N + W, D)).astype(np.float32))
    s0 = torch.from_numpy(rng.random(N).astype(np.float32) + 0.1)
    for S, A in ((V, V), (K, V)):
        got, src, nbr, nbr_e = okv.propagate_unit(A, s0, N, 3, 4, 2, 0.5, Sh=S)
        want, want_src = brute_propagate(S, A, s0, N, 3, 4, 2, 0.5)
        np.testing.assert_allclose(got.numpy(), want, rtol=1e-6)
        assert sorted(src.tolist()) == sorted(want_src.tolist())
        i = int(src[0])
        np.testing.assert_allclose(
            okv.edges_unit(A, N, i, Sh=S).numpy()[nbr[0].numpy()], nbr_e[0].numpy(), rtol=1e-12)


def test_decode_attention_matches_the_library_softmax():
    rng = np.random.default_rng(5)
    q = torch.from_numpy(rng.standard_normal((2, 4, 16)).astype(np.float32) * 2)
    K = torch.from_numpy(rng.standard_normal((2, 2, 37, 16)).astype(np.float32))
    V = torch.from_numpy(rng.standard_normal((2, 2, 37, 16)).astype(np.float32))
    got = okv.decode_attention(q, K, V)
    Kq = K.double().repeat_interleave(2, dim=1)            # KV head h serves query heads 2h, 2h+1
    Vq = V.double().repeat_interleave(2, dim=1)
    P = torch.softmax(torch.einsum("bhd,bhjd->bhj", q.double(), Kq) / 4.0, dim=-1)
    want = torch.einsum("bhj,bhjd->bhd", P, Vq)
    np.testing.assert_allclose(got.numpy(), want.numpy(), rtol=1e-12, atol=1e-14)
    # one cached row: the output is that row's value
    one = okv.decode_attention(q, K[:, :, :1], V[:, :, :1])
    np.testing.assert_allclose(one[0, 3].numpy(), V[0, 1, 0].double().numpy(), rtol=1e-12)
