"""Parity of the multi-token chunk path (tcgen05 kernel, through the C ABI) against the oracle."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from helpers import GpuRunner, assert_close, assert_lse_close

pytestmark = pytest.mark.gpu


def run_chunk(w, **kw):
    K, V, Q = w.make_k(), w.make_v(), w.make_q(0)
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, w.T, w.kv_len, K, V, **kw)
    o, lse, _ = r.run(Q, "chunk")
    o_ref, lse_ref = oracle.xattn(Q, K, V, w.cu, w.kv_len, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=w.T,
                                  scale=kw.get("scale", 0.0))
    res = assert_close(o, o_ref, w.name)
    assert_lse_close(lse, lse_ref, w.name)
    return res


def test_one_tile_no_mask():
    """128 rows x 128 keys, T = 1 per (b, h): a single QK and a single PV product."""
    run_chunk(si.Workload("one_tile", B=32, Hq=4, Hkv=1, d=128, T=1, layers=1, seed=31, kv_len=[128] * 32))


def test_single_stream_causal_block():
    run_chunk(si.Workload("causal", B=1, Hq=1, Hkv=1, d=128, T=128, layers=1, seed=32, kv_len=[128]))


def test_several_key_tiles_and_ragged_tail():
    run_chunk(si.Workload("tail", B=1, Hq=4, Hkv=1, d=128, T=32, layers=1, seed=33, kv_len=[1000]))


def test_chunk_small_config():
    run_chunk(si.workload("chunk_small"))


@pytest.mark.parametrize("Hq,Hkv,T,d,lens", [
    (8, 2, 1, 128, [300, 77]),            # decode-shaped call through the chunk kernel
    (24, 8, 48, 128, [500, 4000]),        # G = 3: row tiles straddle heads
    (4, 4, 300, 64, [300, 1234]),         # d = 64, T not a multiple of 128
    (32, 8, 64, 128, [64, 65]),           # cache holds only (or barely more than) the chunk itself
    (8, 1, 16, 128, [10, 0, 2000]),       # more rows than keys; an empty sequence
])
def test_shapes(Hq, Hkv, T, d, lens):
    run_chunk(si.Workload("shape", B=len(lens), Hq=Hq, Hkv=Hkv, d=d, T=T, layers=1, seed=34, kv_len=lens))


def test_peaked_scores_move_the_reference_max_late():
    w = si.Workload("chunk_peaked", B=1, Hq=8, Hkv=2, d=128, T=64, layers=1, seed=35, kv_len=[6000])
    K, V, Q = w.make_k().reshape(2, 6000, 128).copy(), w.make_v(), w.make_q(0)
    qf = si.bf16_bits_to_f32(Q).reshape(8, 64, 128)
    for c in range(2):
        for n, (pos, gain) in enumerate([(700, 0.5), (3000, 1.0), (5900, 1.5), (5990, 2.0)]):
            K[c, pos] = si.f32_to_bf16_bits(gain * qf[c * 4 + n, 10 * n])
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, w.T, w.kv_len, K, V)
    o, lse, _ = r.run(Q, "chunk")
    o_ref, lse_ref = oracle.xattn(Q, K.reshape(-1), V, w.cu, w.kv_len, B=1, Hq=8, Hkv=2, d=128, T=64)
    assert_close(o, o_ref, "chunk peaked")
    assert_lse_close(lse, lse_ref, "chunk peaked")


def test_capacity_layout_with_nan_slack():
    B, Hq, Hkv, d, T, cap = 1, 8, 2, 128, 40, 512
    lens = np.array([300], dtype=np.int32)
    rng = np.random.default_rng(36)
    K = np.full((Hkv, cap, d), 0x7FC0, dtype=np.uint16)
    V = np.full((Hkv, cap, d), 0x7FC0, dtype=np.uint16)
    K[:, :300] = si.f32_to_bf16_bits(rng.standard_normal((Hkv, 300, d)).astype(np.float32))
    V[:, :300] = si.f32_to_bf16_bits(rng.standard_normal((Hkv, 300, d)).astype(np.float32))
    Q = si.f32_to_bf16_bits(rng.standard_normal((B, Hq, T, d)).astype(np.float32))
    cu = np.array([0, cap], dtype=np.int32)
    r = GpuRunner(B, Hq, Hkv, d, T, lens, K, V, cu=cu, kv_head_stride=cap * d)
    o, lse, _ = r.run(Q, "chunk")
    o_ref, lse_ref = oracle.xattn(Q, K, V, cu, lens, B=B, Hq=Hq, Hkv=Hkv, d=d, T=T, kv_head_stride=cap * d)
    assert_close(o, o_ref, "chunk capacity")
    assert_lse_close(lse, lse_ref, "chunk capacity")


def test_chunk_and_decode_kernels_agree_on_a_small_chunk():
    w = si.Workload("both", B=2, Hq=8, Hkv=2, d=128, T=4, layers=1, seed=37, kv_len=[900, 130])
    K, V, Q = w.make_k(), w.make_v(), w.make_q(0)
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, w.T, w.kv_len, K, V)
    o1, l1, _ = r.run(Q, "chunk")
    o2, l2, _ = r.run(Q, "decode")
    assert np.abs(o1 - o2).max() <= 1e-2 and np.abs(l1 - l2).max() <= 2e-3


def test_two_runs_are_bit_identical():
    import torch
    w = si.workload("chunk_small")
    K, V, Q = w.make_k(), w.make_v(), w.make_q(0)
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, w.T, w.kv_len, K, V)
    _, _, O1 = r.run(Q, "chunk")
    a = O1.clone()
    _, _, O2 = r.run(Q, "chunk")
    assert torch.equal(a.view(torch.int16), O2.view(torch.int16))
