"""Parity of the decode over an 8-bit (FP8 E4M3) cache, through the C ABI, against the oracle
evaluating the same bytes and scales in fp64."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from helpers import GUARD, assert_close, assert_lse_close, bf16_dev_to_f64, to_dev_bf16

pytestmark = pytest.mark.gpu


def run_fp8(w, K8, V8, ks, vs, *, cu=None, stride=0, window=0, layer=0):
    import torch
    from paper_2405_05254_b200 import binding as bd
    Q = w.make_q(layer)
    shape = bd.make_shape(w.B, w.Hq, w.Hkv, w.d, w.T, kv_head_stride=stride, max_kv_len=int(w.kv_len.max()),
                          window=window)
    n = w.B * w.Hq * w.T
    ws = torch.empty(bd.yoco_xattn_workspace_size(shape, w.kv_len, bd.MODE_DECODE), dtype=torch.uint8, device="cuda")
    obuf = torch.full((GUARD + n * w.d + GUARD,), 777.0, dtype=torch.bfloat16, device="cuda")
    O = obuf[GUARD:GUARD + n * w.d]
    L = torch.empty(n, dtype=torch.float32, device="cuda")
    Kd, Vd = torch.from_numpy(K8).cuda(), torch.from_numpy(V8).cuda()
    bd.yoco_xattn_decode_fp8(shape, to_dev_bf16(Q.reshape(-1)), Kd, Vd, ks, vs, cu, w.kv_len, O, L, ws)
    assert bd.yoco_xattn_status(ws) == 0
    assert (obuf[:GUARD] == 777.0).all() and (obuf[-GUARD:] == 777.0).all()
    cu_o = w.cu if cu is None else cu
    o_ref, lse_ref = oracle.xattn_fp8(Q, K8, V8, ks, vs, cu_o, w.kv_len, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=w.T,
                                      kv_head_stride=stride, window=window)
    o = bf16_dev_to_f64(O).reshape(w.B, w.Hq, w.T, w.d)
    assert_close(o, o_ref, w.name)
    assert_lse_close(L.cpu().numpy().reshape(w.B, w.Hq, w.T), lse_ref, w.name)
    return o, o_ref


@pytest.mark.parametrize("Hq,Hkv,T,lens", [
    (32, 8, 1, [1000, 64, 1, 333]),          # the 3B-class head layout, ragged, a one-key sequence
    (8, 2, 2, [500, 65]),                    # two rows per head
    (24, 8, 1, [129, 4000]),                 # G = 3
    (16, 1, 1, [70, 0, 300]),                # 16 rows per KV head (the wide variant), an empty sequence
])
def test_fp8_decode_matches_the_oracle(Hq, Hkv, T, lens):
    w = si.Workload("fp8", B=len(lens), Hq=Hq, Hkv=Hkv, d=128, T=T, layers=1, seed=95, kv_len=lens)
    run_fp8(w, *w.make_kv_fp8())


def test_fp8_decode_long_sequence_is_split_and_merged():
    w = si.Workload("fp8_long", B=1, Hq=32, Hkv=8, d=128, T=1, layers=1, seed=96, kv_len=[40000])
    o, o_ref = run_fp8(w, *w.make_kv_fp8())
    # for context: how far the 8-bit cache is from the bf16 cache it was made from
    ob, _ = oracle.xattn(w.make_q(0), w.make_k(), w.make_v(), w.cu, w.kv_len, B=1, Hq=32, Hkv=8, d=128, T=1)
    assert np.linalg.norm(o_ref - ob) / np.linalg.norm(ob) < 0.1


def test_fp8_decode_with_a_window():
    w = si.Workload("fp8_win", B=2, Hq=8, Hkv=2, d=128, T=1, layers=1, seed=97, kv_len=[3000, 100])
    run_fp8(w, *w.make_kv_fp8(), window=257)


def test_fp8_capacity_layout_with_nan_bytes_in_the_slack():
    """A cache with spare rows per head, the spare bytes set to the E4M3 NaN code: nothing of it
    may reach the result."""
    Hkv, d, cap, n = 2, 128, 256, 150
    w = si.Workload("fp8_cap", B=1, Hq=8, Hkv=Hkv, d=d, T=1, layers=1, seed=98, kv_len=[n])
    K8t, V8t, ks, vs = w.make_kv_fp8()
    K8 = np.full((Hkv, cap, d), 0x7F, dtype=np.uint8)
    V8 = np.full((Hkv, cap, d), 0x7F, dtype=np.uint8)
    K8[:, :n] = K8t.reshape(Hkv, n, d)
    V8[:, :n] = V8t.reshape(Hkv, n, d)
    run_fp8(w, K8.reshape(-1), V8.reshape(-1), ks, vs, cu=np.array([0, cap], np.int32), stride=cap * d)


def test_fp8_entry_rejects_other_head_sizes_and_bad_scales():
    import torch
    from paper_2405_05254_b200 import binding as bd
    t = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    q = torch.zeros(4096, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(bd.YocoError) as e:
        bd.yoco_xattn_decode_fp8(bd.make_shape(1, 1, 1, 64, 1, max_kv_len=8), q, t, t, [1.0], [1.0], None, [8], q, None, t)
    assert e.value.code == bd.ERR_UNSUPPORTED
    with pytest.raises(bd.YocoError) as e:
        bd.yoco_xattn_decode_fp8(bd.make_shape(1, 1, 1, 128, 1, max_kv_len=8), q, t, t, [0.0], [1.0], None, [8], q, None, t)
    assert e.value.code == bd.ERR_INVALID_ARG


def run_chunk_fp8(w, K8, V8, ks, vs, *, cu=None, stride=0, window=0):
    import torch
    from paper_2405_05254_b200 import binding as bd
    Q = w.make_q(0)
    shape = bd.make_shape(w.B, w.Hq, w.Hkv, w.d, w.T, kv_head_stride=stride, max_kv_len=int(w.kv_len.max()),
                          window=window)
    n = w.B * w.Hq * w.T
    ws = torch.empty(bd.yoco_xattn_workspace_size_chunk_fp8(shape, w.kv_len), dtype=torch.uint8, device="cuda")
    obuf = torch.full((GUARD + n * w.d + GUARD,), 777.0, dtype=torch.bfloat16, device="cuda")
    O = obuf[GUARD:GUARD + n * w.d]
    L = torch.empty(n, dtype=torch.float32, device="cuda")
    bd.yoco_xattn_chunk_fp8(shape, to_dev_bf16(Q.reshape(-1)), torch.from_numpy(K8).cuda(), torch.from_numpy(V8).cuda(),
                            ks, vs, cu, w.kv_len, O, L, ws)
    assert bd.yoco_xattn_status(ws) == 0
    assert (obuf[:GUARD] == 777.0).all() and (obuf[-GUARD:] == 777.0).all()
    cu_o = w.cu if cu is None else cu
    o_ref, lse_ref = oracle.xattn_fp8(Q, K8, V8, ks, vs, cu_o, w.kv_len, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=w.T,
                                      kv_head_stride=stride, window=window)
    assert_close(bf16_dev_to_f64(O).reshape(w.B, w.Hq, w.T, w.d), o_ref, w.name)
    assert_lse_close(L.cpu().numpy().reshape(w.B, w.Hq, w.T), lse_ref, w.name)


@pytest.mark.parametrize("Hq,Hkv,T,lens", [
    (32, 8, 160, [1160, 937]),               # the benchmark's head layout: 640 rows per KV head, three CTA row pairs
    (8, 2, 40, [4000, 41]),                  # 160 rows per KV head; a sequence that is all chunk
    (8, 8, 7, [300, 7, 1000]),               # few rows: the second row tile of every CTA is empty
    (24, 8, 64, [129 + 64]),                 # G = 3
    (4, 1, 200, [200, 0, 513]),              # an empty sequence
])
def test_fp8_chunk_matches_the_oracle(Hq, Hkv, T, lens):
    """The tensor-core path reading the 8-bit cache: widened in the kernel, fp16 products."""
    w = si.Workload("fp8_chunk", B=len(lens), Hq=Hq, Hkv=Hkv, d=128, T=T, layers=1, seed=99, kv_len=lens)
    run_chunk_fp8(w, *w.make_kv_fp8())


def test_fp8_chunk_split_over_a_long_cache_with_a_window_and_nan_slack():
    w = si.Workload("fp8_chunk_long", B=1, Hq=32, Hkv=8, d=128, T=96, layers=1, seed=100, kv_len=[20000 + 96])
    K8, V8, ks, vs = w.make_kv_fp8()
    run_chunk_fp8(w, K8, V8, ks, vs)
    run_chunk_fp8(w, K8, V8, ks, vs, window=1000)
    # a cache with spare rows per head holding the E4M3 NaN code
    Hkv, d, n, cap = 2, 128, 333, 512
    w2 = si.Workload("fp8_chunk_cap", B=1, Hq=8, Hkv=Hkv, d=d, T=50, layers=1, seed=101, kv_len=[n])
    K8t, V8t, ks2, vs2 = w2.make_kv_fp8()
    K8c = np.full((Hkv, cap, d), 0x7F, dtype=np.uint8)
    V8c = np.full((Hkv, cap, d), 0x7F, dtype=np.uint8)
    K8c[:, :n] = K8t.reshape(Hkv, n, d)
    V8c[:, :n] = V8t.reshape(Hkv, n, d)
    run_chunk_fp8(w2, K8c.reshape(-1), V8c.reshape(-1), ks2, vs2, cu=np.array([0, cap], np.int32), stride=cap * d)


def test_append_fp8_then_chunk_fp8_reads_what_was_written():
    """The 8-bit cache end to end on the multi-token path: rows written by yoco_kv_append_fp8, read by
    yoco_xattn_chunk_fp8, against the oracle evaluating the bytes the GPU wrote."""
    import torch
    from paper_2405_05254_b200 import binding as bd
    B, T, d_model, Hkv, d, Hq = 1, 200, 512, 2, 128, 8
    X = si.normal_bf16(8, 40, B * T * d_model).reshape(B * T, d_model)
    Wk = si.normal_bf16(8, 42, d_model * Hkv * d, mult=d_model ** -0.5)
    Wv = si.normal_bf16(8, 43, d_model * Hkv * d, mult=d_model ** -0.5)
    lens = np.array([T], dtype=np.int32)
    K8 = torch.zeros(Hkv * T * d, dtype=torch.uint8, device="cuda")
    V8 = torch.zeros_like(K8)
    ks = np.full(Hkv, 6.0 / 448, dtype=np.float32)
    vs = np.full(Hkv, 6.0 / 448, dtype=np.float32)
    bd.yoco_kv_append_fp8(bd.KvAppendShape(B, Hkv, d, T, d_model, 1e-6, 0), to_dev_bf16(X.reshape(-1)),
                          to_dev_bf16(Wk).view(d_model, -1), to_dev_bf16(Wv).view(d_model, -1), K8, V8, ks, vs, None, lens)
    assert bd.yoco_kv_append_status() == 0
    w = si.Workload("fp8_chain", B=B, Hq=Hq, Hkv=Hkv, d=d, T=T, layers=1, seed=102, kv_len=[T])
    run_chunk_fp8(w, K8.cpu().numpy(), V8.cpu().numpy(), ks, vs)


def test_fp8_chunk_at_the_benchmark_row_count_over_a_32k_cache():
    """512 new rows per sequence (2,048 rows per KV head: eight CTA row pairs walking the same keys) after
    32,768 cached keys of an 8-bit cache, every row, against the oracle."""
    w = si.Workload("fp8_chunk_32k", B=1, Hq=32, Hkv=8, d=128, T=512, layers=1, seed=4, kv_len=[32768 + 512])
    run_chunk_fp8(w, *w.make_kv_fp8())
