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
