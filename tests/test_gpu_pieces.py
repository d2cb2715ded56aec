"""The decode path when the plan cuts its groups into work pieces that are handed out at run time
(long caches: 40 key tiles or more per CTA group): parity with the fp64 oracle on ragged batches
with every option the decode call has -- several rows per head, d = 64, a sliding window, a cache
with spare capacity per head -- and the partial-result entry point used by key-range sharding."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from helpers import GpuRunner, assert_close, assert_lse_close, to_dev_bf16

pytestmark = pytest.mark.gpu


def plan_of(w, window=0, stride=0):
    import torch
    from paper_2405_05254_b200 import binding as bd
    sm = torch.cuda.get_device_properties(0).multi_processor_count
    shape = bd.make_shape(w.B, w.Hq, w.Hkv, w.d, w.T, window=window, kv_head_stride=stride,
                          max_kv_len=int(w.kv_len.max()))
    return bd.yoco_xattn_plan(shape, w.kv_len, sm, bd.MODE_DECODE)


@pytest.mark.parametrize("name,kw,pieces", [
    ("two pieces, ragged", dict(B=5, Hq=8, Hkv=8, d=128, T=1, kv_len=[30001, 17, 25000, 40960, 9999]), 2),
    ("four pieces, ragged", dict(B=4, Hq=8, Hkv=8, d=128, T=1, kv_len=[90001, 64, 120000, 31000]), 4),
    ("four pieces, two rows per head, G = 2", dict(B=2, Hq=16, Hkv=8, d=128, T=2, kv_len=[150003, 95000]), 4),
    ("two pieces, d = 64, 16 rows", dict(B=3, Hq=32, Hkv=2, d=64, T=1, kv_len=[200000, 1, 230007]), 2),
    # 200 streams and ~490 segments: too many for the kernel-parameter tables, so the work tables and the
    # work counter live in the workspace
    ("two pieces, tables in the workspace", dict(B=25, Hq=8, Hkv=8, d=128, T=1,
                                                 kv_len=[4000 + 137 * i for i in range(25)]), 2),
])
def test_ragged_batches_in_pieces_match_the_oracle(name, kw, pieces):
    w = si.Workload("pieces", layers=1, seed=31, **kw)
    info, segs = plan_of(w)
    assert info.sub_items == pieces, (info.sub_items, info.total_tiles, info.num_groups)
    K, V, Q = w.make_k(), w.make_v(), w.make_q(0)
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, w.T, w.kv_len, K, V)
    o, lse, _ = r.run(Q)
    o_ref, lse_ref = oracle.xattn(Q, K, V, w.cu, w.kv_len, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=w.T)
    assert_close(o, o_ref, name)
    assert_lse_close(lse, lse_ref, name)


def test_pieces_with_a_sliding_window():
    """The window leaves 2,500 tiles per stream of which the plan keeps those a row can see; the groups
    are still long enough for pieces, and the first kept tile is masked in part."""
    w = si.Workload("pieces_win", B=2, Hq=8, Hkv=8, d=128, T=1, layers=1, seed=32, kv_len=[160000, 140001])
    C = 100000
    info, segs = plan_of(w, window=C)
    assert info.sub_items >= 2 and min(s.k_begin for s in segs if s.b == 0) == (160000 - 1 - C + 1) // 64 * 64
    K, V, Q = w.make_k(), w.make_v(), w.make_q(0)
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, 1, w.kv_len, K, V, window=C)
    o, lse, _ = r.run(Q)
    o_ref, lse_ref = oracle.xattn(Q, K, V, w.cu, w.kv_len, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=1, window=C)
    assert_close(o, o_ref, "pieces + window")
    assert_lse_close(lse, lse_ref, "pieces + window")


def test_pieces_over_a_cache_with_spare_capacity():
    """kv_head_stride > N*d with NaN bit patterns in the slack of every head."""
    B, Hq, Hkv, d, cap = 2, 8, 8, 128, 60032
    lens = np.array([60001, 47000], dtype=np.int32)
    rng = np.random.default_rng(33)
    K = np.full((B, Hkv, cap, d), 0x7FC0, dtype=np.uint16)
    V = np.full((B, Hkv, cap, d), 0x7FC0, dtype=np.uint16)
    for b in range(B):
        n = int(lens[b])
        K[b, :, :n] = si.f32_to_bf16_bits(rng.standard_normal((Hkv, n, d), dtype=np.float32))
        V[b, :, :n] = si.f32_to_bf16_bits(rng.standard_normal((Hkv, n, d), dtype=np.float32))
    Q = si.f32_to_bf16_bits(rng.standard_normal((B, Hq, 1, d), dtype=np.float32))
    cu = np.array([0, cap, 2 * cap], dtype=np.int32)
    r = GpuRunner(B, Hq, Hkv, d, 1, lens, K, V, cu=cu, kv_head_stride=cap * d)
    import torch
    from paper_2405_05254_b200 import binding as bd
    info, _ = bd.yoco_xattn_plan(r.shape, lens, torch.cuda.get_device_properties(0).multi_processor_count, bd.MODE_DECODE)
    assert info.sub_items >= 2
    o, lse, _ = r.run(Q)
    o_ref, lse_ref = oracle.xattn(Q, K, V, cu, lens, B=B, Hq=Hq, Hkv=Hkv, d=d, T=1, kv_head_stride=cap * d)
    assert_close(o, o_ref, "pieces + capacity layout")
    assert_lse_close(lse, lse_ref, "pieces + capacity layout")


def test_partial_entry_point_in_pieces():
    """yoco_xattn_decode_partial over a long shard: fp32 rows and their log-sum-exp equal the oracle's
    attention over that shard alone (a partial result is a complete attention over fewer keys)."""
    import torch
    from paper_2405_05254_b200 import binding as bd
    w = si.Workload("pieces_part", B=1, Hq=32, Hkv=8, d=128, T=1, layers=1, seed=34, kv_len=[131072])
    info, _ = plan_of(w)
    assert info.sub_items == 2
    K, V, Q = w.make_k(), w.make_v(), w.make_q(0)
    shape = bd.make_shape(1, 32, 8, 128, 1, max_kv_len=131072)
    ws = torch.empty(bd.yoco_xattn_workspace_size(shape, w.kv_len, bd.MODE_DECODE), dtype=torch.uint8, device="cuda")
    po = torch.empty(32 * 128, dtype=torch.float32, device="cuda")
    pl = torch.empty(32, dtype=torch.float32, device="cuda")
    bd.yoco_xattn_decode_partial(shape, to_dev_bf16(Q.reshape(-1)), to_dev_bf16(K), to_dev_bf16(V), None, w.kv_len,
                                 po, pl, ws)
    assert bd.yoco_xattn_status(ws) == 0
    o_ref, lse_ref = oracle.xattn(Q, K, V, w.cu, w.kv_len, B=1, Hq=32, Hkv=8, d=128, T=1)
    assert_close(po.cpu().numpy().astype(np.float64).reshape(1, 32, 1, 128), o_ref, "partial in pieces")
    assert_lse_close(pl.cpu().numpy().reshape(1, 32, 1), lse_ref, "partial in pieces")


def test_two_streams_running_pieces_at_once_keep_their_bits():
    """Two long-cache decode problems, each with its own workspace, enqueued on two streams so that their
    grids share the SMs (neither has all its CTAs resident at once): every CTA still runs piece 0 of its
    group whenever it starts, the rest is handed out, and both results stay bit-identical to a solo run."""
    import torch
    from paper_2405_05254_b200 import binding as bd
    probs = []
    for seed, N in ((41, 300000), (42, 180000)):
        w = si.Workload("two", B=1, Hq=32, Hkv=8, d=128, T=1, layers=1, seed=seed, kv_len=[N])
        shape = bd.make_shape(1, 32, 8, 128, 1, max_kv_len=N)
        ws = torch.empty(bd.yoco_xattn_workspace_size(shape, w.kv_len, bd.MODE_DECODE), dtype=torch.uint8, device="cuda")
        probs.append(dict(shape=shape, K=to_dev_bf16(w.make_k()), V=to_dev_bf16(w.make_v()),
                          Q=to_dev_bf16(w.make_q(0).reshape(-1)), lens=w.kv_len, ws=ws,
                          O=torch.empty(32 * 128, dtype=torch.bfloat16, device="cuda")))

    def call(x, stream=None):
        bd.yoco_xattn_decode(x["shape"], x["Q"], x["K"], x["V"], None, x["lens"], x["O"], None, x["ws"], stream)

    for x in probs:
        call(x)
    torch.cuda.synchronize()
    solo = [x["O"].view(torch.int16).clone() for x in probs]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    for _ in range(3):
        for x, s, n in zip(probs, streams, (6, 10)):
            x["O"].zero_()
            with torch.cuda.stream(s):
                for _ in range(n):
                    call(x, s)
        torch.cuda.synchronize()
        for x, ref in zip(probs, solo):
            assert bd.yoco_xattn_status(x["ws"]) == 0
            assert torch.equal(x["O"].view(torch.int16), ref)
