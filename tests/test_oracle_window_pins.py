"""Pins of the oracle's sliding-window mask (Section 3.2: B_ij = 0 iff i - C < j <= i).

None of these re-types the oracle's routine: they use exact special cases (window 1, identical
keys), a reduction to the already pinned unwindowed attention on a cut-down cache, and a dense
mask matrix written from the paper's inequality and fed to a library fp64 softmax.
"""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si

f2b = si.f32_to_bf16_bits
b2f = si.bf16_bits_to_f32


def rnd(rng, *shape):
    return f2b(rng.standard_normal(shape).astype(np.float32))


def call(Q, K, V, kv_len, *, Hkv, window=0, scale=0.0):
    B, Hq, T, d = Q.shape
    kv_len = np.asarray(kv_len, dtype=np.int32)
    cu = np.concatenate([[0], np.cumsum(kv_len)]).astype(np.int32)
    return oracle.xattn(Q, K, V, cu, kv_len, B=B, Hq=Hq, Hkv=Hkv, d=d, T=T, scale=scale, window=window)


def test_window_at_least_the_cache_changes_nothing():
    rng = np.random.default_rng(40)
    Q, K, V = rnd(rng, 2, 4, 3, 8), rnd(rng, (7 + 5) * 2 * 8), rnd(rng, (7 + 5) * 2 * 8)
    O0, L0 = call(Q, K, V, [7, 5], Hkv=2)
    for C in (7, 8, 1000):
        O1, L1 = call(Q, K, V, [7, 5], Hkv=2, window=C)
        np.testing.assert_array_equal(O0, O1)
        np.testing.assert_array_equal(L0, L1)


def test_window_of_one_returns_the_value_at_the_rows_own_position():
    """C = 1 keeps only j = i: O is exactly V[i] and LSE is that single score."""
    rng = np.random.default_rng(41)
    N, T, d = 11, 4, 8
    Q, K, V = rnd(rng, 1, 2, T, d), rnd(rng, N * d), rnd(rng, N * d)
    O, LSE = call(Q, K, V, [N], Hkv=1, window=1)
    Vf, Kf, Qf = (b2f(x).astype(np.float64) for x in (V.reshape(N, d), K.reshape(N, d), Q))
    for t in range(T):
        i = N - T + t
        for h in range(2):
            np.testing.assert_array_equal(O[0, h, t], Vf[i])
            np.testing.assert_allclose(LSE[0, h, t], Qf[0, h, t] @ Kf[i] / np.sqrt(d), rtol=1e-14)


@pytest.mark.parametrize("C", [1, 2, 3, 5, 9, 20])
def test_identical_keys_give_means_over_exactly_the_last_C_positions(C):
    """Equal scores -> uniform weights, so row t is the plain mean of V over (i - C, i]: pins both
    edges of the window for every row, including windows that reach below key 0."""
    rng = np.random.default_rng(42)
    N, T, d = 9, 5, 4
    Q = rnd(rng, 1, 2, T, d)
    K = np.tile(rnd(rng, d), N)
    V = rnd(rng, N * d)
    O, LSE = call(Q, K, V, [N], Hkv=1, window=C)
    Vf = b2f(V).reshape(N, d).astype(np.float64)
    for t in range(T):
        i = N - T + t
        lo = max(0, i - C + 1)
        np.testing.assert_allclose(O[0, 0, t], Vf[lo:i + 1].mean(axis=0), rtol=1e-13, atol=1e-15)
        # LSE = score + log(number of keys in the window)
        s = float(b2f(Q)[0, 0, t].astype(np.float64) @ b2f(K[:d]).astype(np.float64)) / np.sqrt(d)
        np.testing.assert_allclose(LSE[0, 0, t], s + np.log(i + 1 - lo), rtol=1e-13)


def test_decode_row_with_window_equals_full_attention_over_the_last_C_keys():
    """T = 1: a window of C over N keys is plain attention over a cache that holds only keys
    [N - C, N) -- the already pinned unwindowed routine on a cut-down copy."""
    rng = np.random.default_rng(43)
    N, C, d, Hkv, Hq = 37, 10, 16, 2, 6
    Q = rnd(rng, 1, Hq, 1, d)
    K, V = rnd(rng, Hkv, N, d), rnd(rng, Hkv, N, d)
    Ow, Lw = call(Q, K, V, [N], Hkv=Hkv, window=C)
    Oc, Lc = call(Q, np.ascontiguousarray(K[:, N - C:]), np.ascontiguousarray(V[:, N - C:]), [C], Hkv=Hkv)
    np.testing.assert_allclose(Ow, Oc, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(Lw, Lc, rtol=1e-13)


@pytest.mark.parametrize("T,C", [(1, 4), (6, 3), (6, 1), (5, 100), (8, 8)])
def test_dense_mask_from_the_inequality_and_a_library_softmax(T, C):
    """B_ij written out as a dense matrix from i - C < j <= i, applied with torch's fp64 softmax."""
    rng = np.random.default_rng(44)
    B, Hq, Hkv, d = 2, 4, 2, 8
    lens = [13, T]          # the second sequence holds nothing but the chunk itself
    Q = rnd(rng, B, Hq, T, d)
    K, V = rnd(rng, sum(lens) * Hkv * d), rnd(rng, sum(lens) * Hkv * d)
    O, LSE = call(Q, K, V, lens, Hkv=Hkv, window=C)
    off = 0
    for b, N in enumerate(lens):
        Kb = torch.from_numpy(b2f(K[off:off + Hkv * N * d]).reshape(Hkv, N, d).astype(np.float64))
        Vb = torch.from_numpy(b2f(V[off:off + Hkv * N * d]).reshape(Hkv, N, d).astype(np.float64))
        off += Hkv * N * d
        Qb = torch.from_numpy(b2f(Q[b]).astype(np.float64))                    # [Hq, T, d]
        i = torch.arange(N - T, N).view(T, 1)                                  # absolute row positions
        j = torch.arange(N).view(1, N)
        mask = torch.where((i - C < j) & (j <= i), 0.0, -float("inf")).double()
        for h in range(Hq):
            s = Qb[h] @ Kb[h // (Hq // Hkv)].T / np.sqrt(d) + mask
            want = torch.softmax(s, dim=-1) @ Vb[h // (Hq // Hkv)]
            np.testing.assert_allclose(O[b, h], want.numpy(), rtol=1e-12, atol=1e-14)
            np.testing.assert_allclose(LSE[b, h], torch.logsumexp(s, dim=-1).numpy(), rtol=1e-12)


def test_window_commutes_with_split_and_merge():
    rng = np.random.default_rng(45)
    B, Hq, Hkv, d, T, N, C = 1, 4, 2, 8, 3, 40, 11
    Q, K, V = rnd(rng, B, Hq, T, d), rnd(rng, Hkv * N * d), rnd(rng, Hkv * N * d)
    cu, lens = np.array([0, N], dtype=np.int32), np.array([N], dtype=np.int32)
    O, LSE = oracle.xattn(Q, K, V, cu, lens, B=B, Hq=Hq, Hkv=Hkv, d=d, T=T, window=C)
    for cuts in ([20], [5, 28, 30, 35], [29], [0, 39]):
        O2, L2 = oracle.xattn_split_merge(Q, K, V, cu, lens, cuts, B=B, Hq=Hq, Hkv=Hkv, d=d, T=T, window=C)
        np.testing.assert_allclose(O2, O, rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(L2, LSE, rtol=1e-12)


def test_rows_variant_agrees_and_planted_edges_do_not():
    rng = np.random.default_rng(46)
    N, T, d, C = 12, 4, 4, 3
    Q, K, V = rnd(rng, 1, 2, T, d), rnd(rng, N * d), rnd(rng, N * d)
    cu, lens = np.array([0, N], dtype=np.int32), np.array([N], dtype=np.int32)
    O, _ = oracle.xattn(Q, K, V, cu, lens, B=1, Hq=2, Hkv=1, d=d, T=T, window=C)
    rows = np.array([(0, 1, 2), (0, 0, 0)], dtype=np.int32)
    Or, _ = oracle.xattn_rows(Q, K, V, cu, lens, rows, B=1, Hq=2, Hkv=1, d=d, T=T, window=C)
    np.testing.assert_array_equal(Or[0], O[0, 1, 2])
    np.testing.assert_array_equal(Or[1], O[0, 0, 0])
    # a window one key too long or too short (the two plausible off-by-one readings) is a different result
    for wrong in (C - 1, C + 1):
        Ow, _ = oracle.xattn(Q, K, V, cu, lens, B=1, Hq=2, Hkv=1, d=d, T=T, window=wrong)
        assert np.abs(Ow - O).max() > 1e-6
