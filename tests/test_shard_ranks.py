"""Key-range sharding on CPU: the index ranges, the cache slicing, and a world-size-2 gloo run in
which every rank evaluates its own key shard (with the fp64 oracle standing in for the GPU call),
the ranks exchange partial rows through the package's exchange helper, and the merged result is
the unsharded attention."""
import os
import socket
import sys

import numpy as np
import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("lens,world", [([1048576], 8), ([1000, 64, 0, 65, 129], 3), ([5], 4), ([4096] * 4, 2)])
def test_key_ranges_partition_every_sequence_on_tile_boundaries(lens, world):
    from paper_2405_05254_b200 import shard
    off, cnt = shard.key_range_shards(lens, world)
    assert off.shape == cnt.shape == (world, len(lens))
    for i, n in enumerate(lens):
        pos = 0
        for r in range(world):
            assert off[r, i] == pos and cnt[r, i] >= 0
            pos += cnt[r, i]
            if pos < n:
                assert pos % 64 == 0          # only a sequence's last range may end off a tile boundary
        assert pos == n
        nonempty = cnt[:, i][cnt[:, i] > 0]
        if len(nonempty) > 1:
            assert nonempty[:-1].max() - nonempty[:-1].min() == 0 and nonempty[-1] <= nonempty[0]


def test_take_key_range_cuts_the_head_major_layout():
    from paper_2405_05254_b200 import shard
    Hkv, d, lens = 2, 4, [5, 3]
    full = np.arange(sum(lens) * Hkv * d, dtype=np.uint16)
    got = shard.take_key_range(full, lens, Hkv, d, [1, 0], [3, 2])
    seq0 = full[:5 * Hkv * d].reshape(Hkv, 5, d)
    seq1 = full[5 * Hkv * d:].reshape(Hkv, 3, d)
    want = np.concatenate([seq0[:, 1:4].reshape(-1), seq1[:, 0:2].reshape(-1)])
    np.testing.assert_array_equal(got, want)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import oracle
    import synth_inputs as si
    from paper_2405_05254_b200 import shard
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    w = si.Workload("shard_cpu", B=3, Hq=8, Hkv=2, d=16, T=1, layers=1, seed=60, kv_len=[300, 40, 129])
    K, V, Q = w.make_k(), w.make_v(), w.make_q(0)
    off, cnt = shard.key_range_shards(w.kv_len, world)
    Kr = shard.take_key_range(K, w.kv_len, w.Hkv, w.d, off[rank], cnt[rank])
    Vr = shard.take_key_range(V, w.kv_len, w.Hkv, w.d, off[rank], cnt[rank])
    cu = np.concatenate([[0], np.cumsum(cnt[rank])]).astype(np.int32)
    o, lse = oracle.xattn(Q, Kr, Vr, cu, cnt[rank], B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=1)
    part_o = torch.from_numpy(o.reshape(-1, w.d).astype(np.float32))
    part_lse = torch.from_numpy(lse.reshape(-1).astype(np.float32))
    all_o, all_l = shard.exchange_partials(part_o, part_lse)
    assert all_o.shape == (world, w.B * w.Hq, w.d) and all_l.shape == (world, w.B * w.Hq)
    merged, mlse = oracle.combine(all_o.numpy().transpose(1, 0, 2), all_l.numpy().T)
    ref, ref_lse = oracle.xattn(Q, K, V, w.cu, w.kv_len, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=1)
    out.put((rank, float(np.abs(merged - ref.reshape(-1, w.d)).max()),
             float(np.abs(mlse - ref_lse.reshape(-1)).max()), int(cnt[rank].sum())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_each_hold_a_key_range_and_merge_to_the_unsharded_result():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert sum(g[3] for g in got) == 300 + 40 + 129          # every key lives on exactly one rank
    for rank, err_o, err_lse, _ in got:
        assert err_o < 1e-6 and err_lse < 1e-6               # fp32 partials, fp64 merge


def test_exchange_without_a_process_group_adds_a_leading_axis():
    import torch
    from paper_2405_05254_b200 import shard
    o, l = shard.exchange_partials(torch.zeros(4, 8), torch.zeros(4))
    assert o.shape == (1, 4, 8) and l.shape == (1, 4)
