"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The 1M-token (all 13 layers) and ragged decode configs are checked against the full oracle; the
512 x 262K chunk config on at least 64 sampled (sequence, position) query rows, all heads each, over
the full key range (t = 0, T-1, the 128-row tile edges), each computed one by one by the oracle; the
split/merge indexing at 1M tokens bit-exactly with one-hot scores planted on every segment boundary
of the plan; and the side measurements of bench.py at their sizes: the 8-bit cache at 1M keys, a few
new rows per head (the one-tile tensor-core kernel) over a long cache, and one shard of an 8-way
key-range split read through a head-stride view of the resident cache.
"""
import math

import numpy as np
import pytest

import oracle
import synth_inputs as si
from helpers import GpuRunner, assert_close, assert_lse_close, errors, MAX_ABS_TOL, REL_L2_TOL, LSE_ABS_TOL

pytestmark = pytest.mark.gpu


def test_one_million_token_decode_thirteen_layers():
    """Every one of the 13 layer calls over the 1M-token cache, every head, against the full oracle."""
    w = si.workload("1m")
    K, V = w.make_k(), w.make_v()
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, w.T, w.kv_len, K, V)
    kw = dict(B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=w.T)
    for layer in range(w.layers):
        Q = w.make_q(layer)
        o, lse, _ = r.run(Q)
        o_ref, lse_ref = oracle.xattn(Q, K, V, w.cu, w.kv_len, **kw)
        assert_close(o, o_ref, f"1m layer {layer}")
        assert_lse_close(lse, lse_ref, f"1m layer {layer}")


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
    # 36 positions per sequence = 72 (b, t) rows, every head of each: the first and last row, both sides of
    # every 128-row tile edge of the (head in group, t) row order, and seeded draws in between
    edges = [0, 1, 127, 128, 255, 256, 383, 384, 510, 511]
    rng = np.random.default_rng(505)
    inner = [t for t in range(2, 510) if t not in edges]
    ts = sorted(set(edges) | set(int(t) for t in rng.choice(inner, size=26, replace=False)))
    assert len(ts) == 36
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


def test_fp8_cache_decode_at_one_million_tokens():
    """The 8-bit-cache decode at the size bench.py times it, on a really quantised cache (the 1M K/V
    draws rounded to E4M3 with per-head amax / 448 scales), every head, against the oracle reading the
    same bytes."""
    import torch
    from paper_2405_05254_b200 import binding as bd
    from helpers import bf16_dev_to_f64, to_dev_bf16
    w = si.workload("1m")
    K8, V8, ks, vs = w.make_kv_fp8()
    Q = w.make_q(0)
    shape = bd.make_shape(w.B, w.Hq, w.Hkv, w.d, w.T, max_kv_len=int(w.kv_len.max()))
    n = w.B * w.Hq * w.T
    ws = torch.empty(bd.yoco_xattn_workspace_size(shape, w.kv_len, bd.MODE_DECODE), dtype=torch.uint8, device="cuda")
    O = torch.empty(n * w.d, dtype=torch.bfloat16, device="cuda")
    L = torch.empty(n, dtype=torch.float32, device="cuda")
    bd.yoco_xattn_decode_fp8(shape, to_dev_bf16(Q.reshape(-1)), torch.from_numpy(K8).cuda(), torch.from_numpy(V8).cuda(),
                             ks, vs, w.cu, w.kv_len, O, L, ws)
    assert bd.yoco_xattn_status(ws) == 0
    o_ref, lse_ref = oracle.xattn_fp8(Q, K8, V8, ks, vs, w.cu, w.kv_len, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=w.T)
    assert_close(bf16_dev_to_f64(O).reshape(o_ref.shape), o_ref, "fp8 cache, 1M keys")
    assert_lse_close(L.cpu().numpy().reshape(lse_ref.shape), lse_ref, "fp8 cache, 1M keys")


@pytest.mark.parametrize("name", ["ragged", "256k"])
def test_fp8_cache_decode_where_the_plan_cuts_pieces(name):
    """The 8-bit-cache decode on plans with run-time work pieces other than the 1M case: the ragged batch
    (four pieces per group, groups that span several streams, pieces that hold nothing of a segment) and one
    sequence of 262,144 keys (two pieces per group), every head, against the oracle reading the same bytes."""
    import torch
    from paper_2405_05254_b200 import binding as bd
    from helpers import bf16_dev_to_f64, to_dev_bf16
    w = si.workload("ragged") if name == "ragged" else si.Workload("256k", B=1, Hq=32, Hkv=8, d=128, T=1, layers=1,
                                                                      seed=11, kv_len=[262144])
    K8, V8, ks, vs = w.make_kv_fp8()
    Q = w.make_q(0)
    shape = bd.make_shape(w.B, w.Hq, w.Hkv, w.d, w.T, max_kv_len=int(w.kv_len.max()))
    n = w.B * w.Hq * w.T
    ws = torch.empty(bd.yoco_xattn_workspace_size(shape, w.kv_len, bd.MODE_DECODE), dtype=torch.uint8, device="cuda")
    O = torch.empty(n * w.d, dtype=torch.bfloat16, device="cuda")
    L = torch.empty(n, dtype=torch.float32, device="cuda")
    K8d, V8d, Qd = torch.from_numpy(K8).cuda(), torch.from_numpy(V8).cuda(), to_dev_bf16(Q.reshape(-1))
    for _ in range(2):          # the second call finds the workspace as the first one left it
        bd.yoco_xattn_decode_fp8(shape, Qd, K8d, V8d, ks, vs, w.cu, w.kv_len, O, L, ws)
        assert bd.yoco_xattn_status(ws) == 0
    o_ref, lse_ref = oracle.xattn_fp8(Q, K8, V8, ks, vs, w.cu, w.kv_len, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=w.T)
    assert_close(bf16_dev_to_f64(O).reshape(o_ref.shape), o_ref, f"fp8 cache, {name}")
    assert_lse_close(L.cpu().numpy().reshape(lse_ref.shape), lse_ref, f"fp8 cache, {name}")


def test_fp8_chunk_config_sampled_rows_over_the_full_key_range():
    """The multi-token path over the 8-bit cache at the size bench.py times it (2 x 512 new rows after
    262,144 cached keys, a really quantised cache).  The oracle has no row-sampling entry for the 8-bit
    cache, so a sampled row (b, t) is checked as what it is by definition: one query position that sees
    the first N - T + t + 1 keys of its sequence -- a one-row problem over the sequence's part of the
    cache, read in place through a head stride."""
    import torch
    from paper_2405_05254_b200 import binding as bd
    from helpers import bf16_dev_to_f64, to_dev_bf16
    w = si.workload("chunk")
    K8, V8, ks, vs = w.make_kv_fp8()
    Q = w.make_q(0)
    shape = bd.make_shape(w.B, w.Hq, w.Hkv, w.d, w.T, max_kv_len=int(w.kv_len.max()))
    n = w.B * w.Hq * w.T
    ws = torch.empty(bd.yoco_xattn_workspace_size_chunk_fp8(shape, w.kv_len), dtype=torch.uint8, device="cuda")
    O = torch.empty(n * w.d, dtype=torch.bfloat16, device="cuda")
    L = torch.empty(n, dtype=torch.float32, device="cuda")
    bd.yoco_xattn_chunk_fp8(shape, to_dev_bf16(Q.reshape(-1)), torch.from_numpy(K8).cuda(), torch.from_numpy(V8).cuda(),
                            ks, vs, w.cu, w.kv_len, O, L, ws)
    assert bd.yoco_xattn_status(ws) == 0
    o = bf16_dev_to_f64(O).reshape(w.B, w.Hq, w.T, w.d)
    lse = L.cpu().numpy().reshape(w.B, w.Hq, w.T)
    assert np.isfinite(o).all() and np.isfinite(lse).all()
    # the first and last row, both sides of two 128-row tile edges, and seeded draws in between
    rng = np.random.default_rng(506)
    ts = sorted({0, 127, 128, 383, 384, 511} | set(int(t) for t in rng.choice(np.arange(1, 511), size=6, replace=False)))
    per_seq = w.Hkv * w.d
    for b in range(w.B):
        N = int(w.kv_len[b])
        lo, hi = int(w.cu[b]) * per_seq, int(w.cu[b + 1]) * per_seq
        Kb, Vb = K8[lo:hi], V8[lo:hi]                      # [Hkv, N, d] of this sequence
        for t in ts:
            vis = N - w.T + t + 1
            o_ref, lse_ref = oracle.xattn_fp8(Q[b:b + 1, :, t:t + 1, :], Kb, Vb, ks, vs, np.array([0, N], dtype=np.int32),
                                              np.array([vis], dtype=np.int32), B=1, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=1,
                                              kv_head_stride=N * w.d)
            assert_close(o[b, :, t, :], o_ref[0, :, 0, :], f"fp8 chunk row b={b} t={t}")
            assert_lse_close(lse[b, :, t], lse_ref[0, :, 0], f"fp8 chunk row b={b} t={t}")


@pytest.mark.parametrize("T", [8, 32])
def test_few_new_rows_over_a_long_cache(T):
    """T = 8 and 32 new positions per sequence (32 and 128 rows per KV head: the one-tile tensor-core
    kernel, split over the key range and merged) after 131,072 cached keys; every head of sampled
    positions, first and last included, against the oracle row by row."""
    base = si.workload("128k")
    w = si.Workload("few_rows", B=1, Hq=base.Hq, Hkv=base.Hkv, d=base.d, T=T, layers=1, seed=base.seed,
                    kv_len=[131072 + T])
    K, V, Q = w.make_k(), w.make_v(), w.make_q(0)
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, w.T, w.kv_len, K, V)
    o, lse, _ = r.run(Q, "chunk")
    ts = sorted({0, 1, T // 2, T - 2, T - 1} | {3, 5} & set(range(T)))
    rows = np.array([(0, h, t) for t in ts for h in range(w.Hq)], dtype=np.int32)
    o_ref, lse_ref = oracle.xattn_rows(Q, K, V, w.cu, w.kv_len, rows, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=w.T)
    got = np.stack([o[b, h, t] for b, h, t in rows])
    assert_close(got, o_ref, f"T={T} over 131072 keys")
    assert_lse_close(np.array([lse[b, h, t] for b, h, t in rows]), lse_ref, f"T={T} over 131072 keys")
    assert np.isfinite(o).all() and np.isfinite(lse).all()


def test_one_shard_of_an_eight_way_key_split_read_through_a_head_stride_view():
    """What bench.py's key-range-shard measurement runs: the 1M cache stays where it is and a shard is
    the view (pointer offset to its first key, head stride of the whole cache, 131,072 keys per head).
    The partial result of the first, a middle and the last shard against the oracle over the same view,
    and the merge of all eight against the oracle over the whole cache."""
    import torch
    from paper_2405_05254_b200 import binding as bd, shard
    from helpers import bf16_dev_to_f64, to_dev_bf16
    w = si.workload("1m")
    K, V, Q = w.make_k(), w.make_v(), w.make_q(0)
    N, shards = int(w.kv_len[0]), 8
    off, cnt = shard.key_range_shards([N], shards)
    Kd, Vd, Qd = to_dev_bf16(K), to_dev_bf16(V), to_dev_bf16(Q.reshape(-1))
    rows = w.B * w.Hq
    all_o = torch.zeros((shards, rows, w.d), dtype=torch.float32, device="cuda")
    all_l = torch.zeros((shards, rows), dtype=torch.float32, device="cuda")
    cu = np.array([0, N], dtype=np.int32)
    for r in range(shards):
        n_local = int(cnt[r, 0])
        assert n_local == 131072
        lens = np.array([n_local], dtype=np.int32)
        shape = bd.make_shape(1, w.Hq, w.Hkv, w.d, 1, kv_head_stride=N * w.d, max_kv_len=n_local)
        ws = torch.empty(bd.yoco_xattn_workspace_size(shape, lens, bd.MODE_DECODE), dtype=torch.uint8, device="cuda")
        o = int(off[r, 0]) * w.d
        bd.yoco_xattn_decode_partial(shape, Qd, Kd[o:], Vd[o:], cu, lens, all_o[r], all_l[r], ws)
        assert bd.yoco_xattn_status(ws) == 0
        if r in (0, 3, 7):
            po, pl = oracle.xattn(Q, K[o:], V[o:], cu, lens, B=1, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=1, kv_head_stride=N * w.d)
            got = all_o[r].cpu().numpy().astype(np.float64).reshape(po.shape)
            assert_close(got, po, f"shard {r}")
            assert_lse_close(all_l[r].cpu().numpy().reshape(pl.shape), pl, f"shard {r}")
    O = torch.empty(rows * w.d, dtype=torch.bfloat16, device="cuda")
    L = torch.empty(rows, dtype=torch.float32, device="cuda")
    bd.yoco_xattn_combine_gathered(all_o, all_l, O, L)
    torch.cuda.synchronize()
    o_ref, lse_ref = oracle.xattn(Q, K, V, w.cu, w.kv_len, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=w.T)
    assert_close(bf16_dev_to_f64(O).reshape(o_ref.shape), o_ref, "eight shards merged")
    assert_lse_close(L.cpu().numpy().reshape(lse_ref.shape), lse_ref, "eight shards merged")
