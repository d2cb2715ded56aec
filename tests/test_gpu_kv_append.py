"""Parity of the cache-writing step (K^ = RMSNorm(X) W_K, V^ = RMSNorm(X) W_V appended head-major)
through the C ABI against the fp64 oracle, and the end-to-end check that attention over a cache
written by the GPU matches the oracle's attention over the oracle's cache."""
import numpy as np
import pytest

import synth_inputs as si
from helpers import REL_L2_TOL, bf16_dev_to_f64, errors, to_dev_bf16
from oracle import kv_append as ka

pytestmark = pytest.mark.gpu
SENTINEL = 0x4F80          # bf16 bits of 2^32: untouched cache rows must keep it


def make_inputs(seed, B, T, d_model, Hkv, d):
    n_out = Hkv * d
    X = si.normal_bf16(seed, 40, B * T * d_model).reshape(B * T, d_model)
    g = si.f32_to_bf16_bits(1.0 + 0.25 * si.bf16_bits_to_f32(si.normal_bf16(seed, 41, d_model)))
    Wk = si.normal_bf16(seed, 42, d_model * n_out, mult=d_model ** -0.5).reshape(d_model, n_out)
    Wv = si.normal_bf16(seed, 43, d_model * n_out, mult=d_model ** -0.5).reshape(d_model, n_out)
    return X, g, Wk, Wv


def run_append(seed, B, T, d_model, Hkv, d, lens, eps=1e-6, cap=0):
    import torch
    from paper_2405_05254_b200 import binding as bd
    X, g, Wk, Wv = make_inputs(seed, B, T, d_model, Hkv, d)
    lens = np.asarray(lens, dtype=np.int32)
    if cap:
        cu = (np.arange(B + 1) * cap).astype(np.int32)
        stride, total_rows = cap * d, B * Hkv * cap
    else:
        cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
        stride, total_rows = 0, int(lens.sum()) * Hkv
    K = torch.from_numpy(np.full(total_rows * d, SENTINEL, np.uint16).view(np.int16)).cuda().view(torch.bfloat16)
    V = K.clone()
    Wgk = torch.empty((d_model, Hkv * d), dtype=torch.bfloat16, device="cuda")
    Wgv = torch.empty_like(Wgk)
    gd = to_dev_bf16(g)
    bd.yoco_kv_fold_gain(gd, to_dev_bf16(Wk).view(d_model, -1), Wgk)
    bd.yoco_kv_fold_gain(gd, to_dev_bf16(Wv).view(d_model, -1), Wgv)
    # the fold is one exact product and one rounding: bit for bit
    want = si.f32_to_bf16_bits(si.bf16_bits_to_f32(g)[:, None] * si.bf16_bits_to_f32(Wk))
    assert np.array_equal(Wgk.view(torch.int16).cpu().numpy().view(np.uint16), want)
    shape = bd.KvAppendShape(B, Hkv, d, T, d_model, eps, stride)
    bd.yoco_kv_append(shape, to_dev_bf16(X.reshape(-1)), Wgk, Wgv, K, V, cu if cap else None, lens)
    assert bd.yoco_kv_append_status() == 0
    off, Kr, Vr = ka.kv_append(X, g, Wk, Wv, B=B, Hkv=Hkv, d=d, T=T, cu=cu, kv_len=lens, eps=eps, kv_head_stride=stride)
    Kh, Vh = bf16_dev_to_f64(K), bf16_dev_to_f64(V)
    written = np.zeros(total_rows * d, dtype=bool)
    for name, got_all, ref in (("K", Kh, Kr), ("V", Vh, Vr)):
        got = np.stack([[got_all[o:o + d] for o in row] for row in off])       # [B*T, Hkv, d]
        max_abs, rel_l2 = errors(got, ref)
        assert np.isfinite(got).all() and rel_l2 <= REL_L2_TOL and max_abs <= 1e-2 * max(1.0, np.abs(ref).max()), \
            (name, max_abs, rel_l2)
    for o in off.reshape(-1):
        written[o:o + d] = True
    raw = K.view(torch.int16).cpu().numpy().view(np.uint16)
    assert (raw[~written] == SENTINEL).all(), "rows outside the appended positions were touched"
    return K, V, (X, g, Wk, Wv), cu, lens


@pytest.mark.parametrize("B,T,d_model,Hkv,d,lens", [
    (1, 128, 128, 1, 128, [128]),                 # one tile, one K step
    (2, 1, 4096, 8, 128, [300, 1]),               # decode: one new token per sequence
    (3, 40, 3072, 8, 128, [40, 1000, 77]),        # the paper's width, tokens straddle tiles and sequences
    (2, 200, 1024, 2, 64, [200, 513]),            # d = 64: one output tile covers two heads
    (16, 1, 512, 4, 128, list(range(1, 17))),     # a row of the tile per sequence
])
def test_append_matches_the_oracle_and_touches_nothing_else(B, T, d_model, Hkv, d, lens):
    run_append(80, B, T, d_model, Hkv, d, lens)


def test_append_into_a_cache_with_spare_capacity_and_another_eps():
    run_append(81, 2, 9, 1024, 8, 128, [100, 9], eps=1e-2, cap=128)


def test_attention_over_a_cache_written_on_the_gpu():
    """Prefill chunk end to end: the GPU writes the T new rows, the chunk kernel attends over
    them; the oracle does both steps in fp64 (its own cache rounded to bf16 as the format demands)."""
    import oracle
    from paper_2405_05254_b200 import binding as bd
    import torch
    B, T, d_model, Hkv, d, Hq = 1, 256, 1024, 2, 128, 8
    K, V, (X, g, Wk, Wv), cu, lens = run_append(82, B, T, d_model, Hkv, d, [T])
    Q = si.normal_bf16(82, 44, B * Hq * T * d).reshape(B, Hq, T, d)
    shape = bd.make_shape(B, Hq, Hkv, d, T, max_kv_len=T)
    ws = torch.empty(bd.yoco_xattn_workspace_size(shape, lens, bd.MODE_CHUNK), dtype=torch.uint8, device="cuda")
    O = torch.empty(B * Hq * T * d, dtype=torch.bfloat16, device="cuda")
    bd.yoco_xattn_chunk(shape, to_dev_bf16(Q.reshape(-1)), K, V, None, lens, O, None, ws)
    assert bd.yoco_xattn_status(ws) == 0
    _, Kr, Vr = ka.kv_append(X, g, Wk, Wv, B=B, Hkv=Hkv, d=d, T=T, cu=cu, kv_len=lens)
    to_cache = lambda r: si.f32_to_bf16_bits(r.transpose(1, 0, 2).astype(np.float32))   # [Hkv, T, d]  # noqa: E731
    o_ref, _ = oracle.xattn(Q, to_cache(Kr), to_cache(Vr), cu, lens, B=B, Hq=Hq, Hkv=Hkv, d=d, T=T)
    max_abs, rel_l2 = errors(bf16_dev_to_f64(O).reshape(B, Hq, T, d), o_ref)
    assert max_abs <= 2e-2 and rel_l2 <= 2 * REL_L2_TOL, (max_abs, rel_l2)
