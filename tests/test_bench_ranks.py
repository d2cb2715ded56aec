"""The N > 1 plumbing of bench.py on CPU: two gloo ranks agree on the slowest time, the job value
sums the replicas' work, and the reference arm runs on rank 0 only."""
import json
import os
import socket
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    from paper_2405_05254_b200 import ranks
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    assert ranks.dist_env() == (rank, rank, world)
    mine = [10.0 + 5.0 * rank, 3.0 - rank]          # rank 1 is slower on the first, faster on the second
    slowest = ranks.max_over_ranks(mine)
    value = ranks.job_throughput_gbs(1_000_000_000, 13, world, slowest[0])
    out.put((rank, slowest, value, ranks.replica_seed(3, rank)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_time_and_sum_the_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, value, seed in got:
        assert slowest == [15.0, 3.0]
        assert abs(value - 2 * 13 * 1e9 / 15e-3 / 1e9) < 1e-6
    assert [g[3] for g in got] == [3, 1003]          # distinct cache contents per replica


def _shard_worker(rank, world, port, out):
    """One rank of the key-range-sharded bench mode on CPU: its share of the keys, the exchange of the
    partial rows through the same helper the GPU mode uses, the slowest rank's time, the job line."""
    import numpy as np
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    import synth_inputs as si
    from paper_2405_05254_b200 import ranks, shard
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    w = si.workload("1m")
    N = int(w.kv_len[0])
    off, cnt = shard.key_range_shards([N], world)
    rows = w.B * w.Hq
    part_o = torch.full((rows, w.d), float(rank + 1))
    part_l = torch.full((rows,), float(10 * (rank + 1)))
    all_o, all_l = shard.exchange_partials(part_o, part_l)
    my_ms = 100.0 + 50.0 * rank                                 # rank 1 is the slow one
    total_ms = ranks.max_over_ranks([my_ms])[0]
    line = bench.shard_keys_line(w, world, steps=4, warmup=3, total_ms=total_ms, clocks=None,
                                 exchange_bytes=rows * (w.d + 1) * 4)
    out.put((rank, int(off[rank, 0]), int(cnt[rank, 0]), tuple(all_o[:, 0, 0].tolist()), tuple(all_l[:, 0].tolist()),
             total_ms, json.dumps(line)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_of_the_key_sharded_mode():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_shard_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [(g[1], g[2]) for g in got] == [(0, 524288), (524288, 524288)]      # the two halves of the 1M keys
    for rank, _, _, gathered_o, gathered_l, total_ms, line in got:
        assert gathered_o == (1.0, 2.0) and gathered_l == (10.0, 20.0)          # rank-major, as the merge reads it
        assert total_ms == 150.0                                               # the slowest rank
        line = json.loads(line)
        assert line["n_gpus"] == 2 and line["scaling"] == "strong" and line["mode"] == "shard-keys"
        # the WHOLE cache once per layer call over the slowest rank's time: 4 steps x 13 layers x 4 GiB / 0.15 s
        assert abs(line["value"] - 4 * 13 * 4294967296 / 0.150 / 1e9) < 1e-6
        assert abs(line["ms_per_step"] - 37.5) < 1e-9 and line["exchange_bytes_per_rank_per_call"] == 32 * 129 * 4


def test_single_process_max_is_identity():
    from paper_2405_05254_b200 import ranks
    assert ranks.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "tiny", "--steps", "2", "--warmup", "1"], env=env, capture_output=True,
                       text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "tiny", "--steps", "2", "--warmup", "1"], env=env, capture_output=True,
                       text=True, timeout=300)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
