"""Pins of the cache-writing oracle (K^ = LN(X) W_K, V^ = LN(X) W_V with RMSNorm, Section 2.2).

Closed forms, invariances, a library routine (torch's fp64 rms_norm + matmul) and a layout check
with one-hot weights; no test re-types the oracle's own expression with the same calls.
"""
import numpy as np
import torch

import synth_inputs as si
from oracle import kv_append as ka

f2b = si.f32_to_bf16_bits
b2f = si.bf16_bits_to_f32


def rnd(rng, *shape, mult=1.0):
    return f2b((mult * rng.standard_normal(shape)).astype(np.float32))


def test_constant_row_normalises_to_signed_ones():
    """x = (a, a, ..., a): mean square a^2, so with eps = 0 the normalised row is sign(a) everywhere
    and K^ is sign(a) times the column sums of g-scaled W."""
    rng = np.random.default_rng(70)
    dm, n = 16, 8
    X = f2b(np.stack([np.full(dm, 3.0), np.full(dm, -0.5)]).astype(np.float32))
    g, Wk, Wv = rnd(rng, dm), rnd(rng, dm, n), rnd(rng, dm, n)
    Kr, Vr = ka.kv_rows(X, g, Wk, Wv, eps=0.0)
    gk = b2f(g).astype(np.float64)[:, None] * b2f(Wk).astype(np.float64)
    np.testing.assert_allclose(Kr[0], gk.sum(axis=0), rtol=1e-13)
    np.testing.assert_allclose(Kr[1], -gk.sum(axis=0), rtol=1e-13)


def test_one_hot_row_picks_one_weight_row_times_sqrt_width():
    """x = a * e_k: mean square a^2 / d_model, so LN(x) = sign(a) sqrt(d_model) g_k e_k and the
    product is that multiple of row k of W."""
    rng = np.random.default_rng(71)
    dm, n, k = 16, 8, 5
    x = np.zeros((1, dm), dtype=np.float32)
    x[0, k] = -2.0
    g, Wk, Wv = rnd(rng, dm), rnd(rng, dm, n), rnd(rng, dm, n)
    Kr, Vr = ka.kv_rows(f2b(x), g, Wk, Wv, eps=0.0)
    scale = -np.sqrt(dm) * float(b2f(g)[k])
    np.testing.assert_allclose(Vr[0], scale * b2f(Wv)[k].astype(np.float64), rtol=1e-13)
    np.testing.assert_allclose(Kr[0], scale * b2f(Wk)[k].astype(np.float64), rtol=1e-13)


def test_invariances_scale_of_x_gain_and_weights():
    rng = np.random.default_rng(72)
    dm, n, M = 32, 16, 5
    X, g, Wk, Wv = rnd(rng, M, dm), rnd(rng, dm), rnd(rng, dm, n), rnd(rng, dm, n)
    K0, V0 = ka.kv_rows(X, g, Wk, Wv, eps=0.0)
    # powers of two are exact in bf16: 4x leaves LN(x) unchanged, 2g and 2W double the result
    X4 = f2b(4.0 * b2f(X))
    K1, _ = ka.kv_rows(X4, g, Wk, Wv, eps=0.0)
    np.testing.assert_allclose(K1, K0, rtol=1e-13)
    K2, V2 = ka.kv_rows(X, f2b(2.0 * b2f(g)), Wk, f2b(2.0 * b2f(Wv)), eps=0.0)
    np.testing.assert_allclose(K2, 2.0 * K0, rtol=1e-13)
    np.testing.assert_allclose(V2, 4.0 * V0, rtol=1e-13)
    # eps matters exactly as the definition says: a huge eps kills the output
    K3, _ = ka.kv_rows(X, g, Wk, Wv, eps=1e12)
    assert np.abs(K3).max() < 1e-4 * np.abs(K0).max()


def test_library_rms_norm_and_matmul():
    rng = np.random.default_rng(73)
    dm, n, M = 64, 24, 7
    X, g, Wk, Wv = rnd(rng, M, dm), rnd(rng, dm), rnd(rng, dm, n), rnd(rng, dm, n)
    for eps in (1e-6, 1e-2):
        Kr, Vr = ka.kv_rows(X, g, Wk, Wv, eps=eps)
        t = lambda a: torch.from_numpy(b2f(a).astype(np.float64))  # noqa: E731
        xn = torch.nn.functional.rms_norm(t(X), (dm,), weight=t(g), eps=eps)
        np.testing.assert_allclose(Kr, (xn @ t(Wk)).numpy(), rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(Vr, (xn @ t(Wv)).numpy(), rtol=1e-12, atol=1e-14)


def test_rows_land_at_the_last_T_positions_of_each_sequence_and_head():
    """Weights that copy channel k of the normalised row to output column k tag every output
    element with where it came from; the offsets must be those of (i, c, N_i - T + t, e) in the
    packed head-major layout, for tight packing and for a cache with spare capacity per head."""
    B, Hkv, d, T = 3, 2, 4, 2
    dm = Hkv * d
    lens = np.array([5, 2, 9], dtype=np.int32)
    for stride, cu in ((0, np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)),
                       (16 * d, np.array([0, 16, 32, 48], dtype=np.int32))):
        off, Kr, Vr = ka.kv_append(np.zeros((B * T, dm), np.uint16), np.zeros(dm, np.uint16),
                                   np.zeros((dm, dm), np.uint16), np.zeros((dm, dm), np.uint16),
                                   B=B, Hkv=Hkv, d=d, T=T, cu=cu, kv_len=lens, kv_head_stride=stride)
        assert off.shape == (B * T, Hkv) and Kr.shape == (B * T, Hkv, d)
        for i in range(B):
            head_rows = stride // d if stride else int(lens[i])
            for t in range(T):
                for c in range(Hkv):
                    want = (int(cu[i]) * Hkv + c * head_rows + int(lens[i]) - T + t) * d
                    assert off[i * T + t, c] == want
        assert len(set(off.reshape(-1).tolist())) == off.size          # no two rows collide


def test_planted_mistakes_are_caught():
    """Gain applied before the normalisation statistic, a transposed weight, or mean replaced by
    sum are different functions: the pins above would see them."""
    rng = np.random.default_rng(74)
    dm, M = 8, 3
    X, g, W = rnd(rng, M, dm), rnd(rng, dm), rnd(rng, dm, dm)
    K0, _ = ka.kv_rows(X, g, W, W, eps=0.0)
    Xf, gf, Wf = (b2f(a).astype(np.float64) for a in (X, g, W))
    wrong_gain_first = ((Xf * gf) / np.sqrt(((Xf * gf) ** 2).mean(axis=1, keepdims=True))) @ Wf
    wrong_transposed = (Xf / np.sqrt((Xf ** 2).mean(axis=1, keepdims=True)) * gf) @ Wf.T
    wrong_sum = (Xf / np.sqrt((Xf ** 2).sum(axis=1, keepdims=True)) * gf) @ Wf
    for wrong in (wrong_gain_first, wrong_transposed, wrong_sum):
        assert np.abs(wrong - K0).max() > 1e-3
