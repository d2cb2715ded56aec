"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The 1M-token and ragged decode configs are checked against the full oracle (one or two layers
completely, the other layers on sampled heads); the 512 x 262K chunk config on sampled query
rows over the full key range (t = 0, T-1, the 128-row tile edges), each computed one by one by
the oracle; and the split/merge indexing at 1M tokens bit-exactly with one-hot scores planted on
every segment boundary of the plan.
"""
import math

import numpy as np
import pytest

import oracle
import synth_inputs as si
from helpers import GpuRunner, assert_close, assert_lse_close, errors, MAX_ABS_TOL, REL_L2_TOL, LSE_ABS_TOL

pytestmark = pytest.mark.gpu


def test_one_million_token_decode_thirteen_layers():
    w = si.workload("1m")
    K, V = w.make_k(), w.make_v()
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, w.T, w.kv_len, K, V)
    kw = dict(B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=w.T)
    for layer in range(w.layers):
        Q = w.make_q(layer)
        o, lse, _ = r.run(Q)
        if layer in (0, w.layers - 1):
            o_ref, lse_ref = oracle.xattn(Q, K, V, w.cu, w.kv_len, **kw)
            assert_close(o, o_ref, f"1m layer {layer}")
            assert_lse_close(lse, lse_ref, f"1m layer {layer}")
        else:   # two query heads of different KV heads, chosen by layer
            heads = [(3 * layer) % w.Hq, (3 * layer + 17) % w.Hq]
            rows = np.array([(0, h, 0) for h in heads], dtype=np.int32)
            o_ref, lse_ref = oracle.xattn_rows(Q, K, V, w.cu, w.kv_len, rows, **kw)
            got = np.stack([o[0, h, 0] for h in heads])
            assert_close(got, o_ref, f"1m layer {layer} heads {heads}")
            assert_lse_close(np.array([lse[0, h, 0] for h in heads]), lse_ref, f"1m layer {layer}")


def test_ragged_batch_full_size():
    w = si.workload("ragged")
    K, V, Q = w.make_k(), w.make_v(), w.make_q(0)
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, w.T, w.kv_len, K, V)
    o, lse, _ = r.run(Q)
    o_ref, lse_ref = oracle.xattn(Q, K, V, w.cu, w.kv_len, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=w.T)
    assert_close(o, o_ref, "ragged")
    assert_lse_close(lse, lse_ref, "ragged")
    for b in range(w.B):                       # per sequence as well: short ones must not hide
        assert_close(o[b], o_ref[b], f"ragged seq {b}")


def test_chunk_config_sampled_rows_over_the_full_key_range():
    w = si.workload("chunk")
    K, V, Q = w.make_k(), w.make_v(), w.make_q(0)
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, w.T, w.kv_len, K, V)
    o, lse, _ = r.run(Q, "chunk")
    ts = [0, 1, 127, 128, 255, 256, 383, 384, 510, 511, 77, 300]
    rows = np.array([(b, h, t) for b in range(w.B) for t in ts for h in range(w.Hq)], dtype=np.int32)
    o_ref, lse_ref = oracle.xattn_rows(Q, K, V, w.cu, w.kv_len, rows, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=w.T)
    got = np.stack([o[b, h, t] for b, h, t in rows])
    assert_close(got, o_ref, "chunk sampled rows")
    assert_lse_close(np.array([lse[b, h, t] for b, h, t in rows]), lse_ref, "chunk sampled rows")
    # properties that hold for every row: finite, and each channel inside the range of V
    assert np.isfinite(o).all() and np.isfinite(lse).all()
    assert np.abs(o).max() <= si.bf16_bits_to_f32(V).max() + 1e-2


def test_split_merge_indexing_is_bit_exact_at_one_million_tokens():
    """One key per KV head leads by > 1000 nats, so fp32 gives it weight exactly 1 and the output
    must equal that key's V row bit for bit.  The key is planted on the first and last position of
    every segment of the 1M plan (the seams of the split/merge), two segments per launch."""
    import torch
    from paper_2405_05254_b200 import binding as bd
    w = si.workload("1m")
    N, Hkv, d, Hq = int(w.kv_len[0]), w.Hkv, w.d, w.Hq
    V = w.make_v()
    shape = bd.make_shape(1, Hq, Hkv, d, 1)
    sm = torch.cuda.get_device_properties(0).multi_processor_count
    info, segs = bd.yoco_xattn_plan(shape, w.kv_len, sm, bd.MODE_DECODE)
    per_head = {c: sorted({x for s in segs if s.c == c for x in (s.k_begin, s.k_end - 1)}) for c in range(Hkv)}
    rounds = max(len(v) for v in per_head.values())
    r = GpuRunner(1, Hq, Hkv, d, 1, w.kv_len, np.zeros(w.kv_elems, dtype=np.uint16), V)
    Kd = r.K.view(Hkv, N, d)
    hot = torch.full((d,), 8.0, dtype=torch.bfloat16, device="cuda")
    Q = si.f32_to_bf16_bits(np.full((1, Hq, 1, d), 16.0, dtype=np.float32))
    Vf = si.bf16_bits_to_f32(V).reshape(Hkv, N, d)
    G = Hq // Hkv
    for k in range(rounds):
        picks = [per_head[c][k % len(per_head[c])] for c in range(Hkv)]
        for c in range(Hkv):
            Kd[c, picks[c]] = hot
        o, lse, _ = r.run(Q)
        for c in range(Hkv):
            Kd[c, picks[c]] = 0
        for h in range(Hq):
            np.testing.assert_array_equal(o[0, h, 0], Vf[h // G, picks[h // G]].astype(np.float64),
                                          err_msg=f"round {k} head {h} key {picks[h // G]}")
        assert np.allclose(lse, 16 * 8 * d / math.sqrt(d), rtol=1e-6)
