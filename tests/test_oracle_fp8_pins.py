"""Pins of the oracle's 8-bit (FP8 E4M3) cache path and of the synthetic quantiser that feeds it."""
import numpy as np
import pytest

import oracle
import synth_inputs as si


def test_e4m3_decoder_on_values_fixed_by_the_format():
    # sign | 4-bit exponent (bias 7) | 3-bit mantissa; exponent 0 subnormal; S.1111.111 NaN; max 448
    known = {0x00: 0.0, 0x01: 2.0 ** -9, 0x07: 7 * 2.0 ** -9, 0x08: 2.0 ** -6, 0x38: 1.0, 0x39: 1.125,
             0x3C: 1.5, 0x40: 2.0, 0x77: 240.0, 0x78: 256.0, 0x7E: 448.0, 0xB8: -1.0, 0xC0: -2.0, 0xFE: -448.0}
    for code, val in known.items():
        assert oracle.e4m3_to_f64(code) == val
    assert np.isnan(oracle.e4m3_to_f64(0x7F)) and np.isnan(oracle.e4m3_to_f64(0xFF))
    vals = [oracle.e4m3_to_f64(c) for c in range(0x7F)]
    assert all(b > a for a, b in zip(vals, vals[1:]))          # codes 0x00..0x7E ascend strictly


def test_two_independent_decoders_agree_on_all_codes_and_the_quantiser_round_trips():
    tab = si.e4m3_table()
    for c in range(256):
        a, b = oracle.e4m3_to_f64(c), tab[c]
        assert (np.isnan(a) and np.isnan(b)) or (a == b and np.signbit(a) == np.signbit(b))
    finite = np.array([c for c in range(256) if c not in (0x7F, 0xFF)])
    np.testing.assert_array_equal(si.quantize_e4m3(tab[finite]), finite.astype(np.uint8))
    # nearest with ties to even, saturation
    assert si.quantize_e4m3(np.array([1.0625]))[0] == 0x38      # halfway 1.0 / 1.125 -> even mantissa (1.0)
    assert si.quantize_e4m3(np.array([1.1875]))[0] == 0x3A      # halfway 1.125 / 1.25 -> 1.25
    assert si.quantize_e4m3(np.array([1e9, -1e9])).tolist() == [0x7E, 0xFE]
    assert si.quantize_e4m3(np.array([1.06, 1.07])).tolist() == [0x38, 0x39]


def test_fp8_cache_with_values_exact_in_both_formats_equals_the_bf16_path():
    """Small integers and halves are exact in E4M3 and in bf16: with power-of-two scales the two
    cache formats describe the same numbers, so the two oracle paths must agree to rounding."""
    rng = np.random.default_rng(90)
    B, Hq, Hkv, d, T, lens = 2, 4, 2, 8, 3, [9, 4]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    n = sum(lens) * Hkv * d
    kvals, vvals = rng.integers(-6, 7, n) / 2.0, rng.integers(-8, 9, n) / 4.0
    Q = si.f32_to_bf16_bits(rng.standard_normal((B, Hq, T, d)).astype(np.float32))
    K8, V8 = si.quantize_e4m3(kvals), si.quantize_e4m3(vvals)
    ks, vs = np.array([2.0, 0.5], np.float32), np.array([0.25, 4.0], np.float32)
    # the bf16 cache holds scale * value, head by head
    def scaled(vals, sc):
        out, off = np.empty(n, np.float32), 0
        for L in lens:
            blk = vals[off:off + Hkv * L * d].reshape(Hkv, L, d) * sc[:, None, None]
            out[off:off + Hkv * L * d] = blk.reshape(-1)
            off += Hkv * L * d
        return si.f32_to_bf16_bits(out)
    O8, L8 = oracle.xattn_fp8(Q, K8, V8, ks, vs, cu, lens, B=B, Hq=Hq, Hkv=Hkv, d=d, T=T)
    Ob, Lb = oracle.xattn(Q, scaled(kvals, ks), scaled(vvals, vs), cu, lens, B=B, Hq=Hq, Hkv=Hkv, d=d, T=T)
    np.testing.assert_allclose(O8, Ob, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(L8, Lb, rtol=1e-13)


def test_scales_act_as_the_definition_says():
    """Doubling v_scale doubles O; multiplying k_scale by a equals multiplying the softmax scale by a."""
    w = si.Workload("fp8pin", B=1, Hq=4, Hkv=2, d=16, T=2, layers=1, seed=91, kv_len=[20])
    K8, V8, ks, vs = w.make_kv_fp8()
    Q = w.make_q(0)
    kw = dict(B=1, Hq=4, Hkv=2, d=16, T=2)
    O, L = oracle.xattn_fp8(Q, K8, V8, ks, vs, w.cu, w.kv_len, **kw)
    O2, L2 = oracle.xattn_fp8(Q, K8, V8, ks, 2 * vs, w.cu, w.kv_len, **kw)
    np.testing.assert_allclose(O2, 2 * O, rtol=1e-14)
    np.testing.assert_array_equal(L2, L)
    O3, L3 = oracle.xattn_fp8(Q, K8, V8, 4 * ks, vs, w.cu, w.kv_len, **kw)
    O4, L4 = oracle.xattn_fp8(Q, K8, V8, ks, vs, w.cu, w.kv_len, scale=4 / np.sqrt(16), **kw)
    np.testing.assert_allclose(O3, O4, rtol=1e-12)
    np.testing.assert_allclose(L3, L4, rtol=1e-12)
    # the quantised cache stays close to the bf16 one it came from (3 mantissa bits: a few percent)
    Ob, _ = oracle.xattn(Q, w.make_k(), w.make_v(), w.cu, w.kv_len, **kw)
    assert np.linalg.norm(O - Ob) / np.linalg.norm(Ob) < 0.1
