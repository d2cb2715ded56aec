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
