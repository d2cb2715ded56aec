"""Host-side plumbing for running independent replicas on several GPUs (one process per GPU).

The attention path shards by replica (each rank owns its own K/V cache and its own calls), so
there is no data-path collective: ranks only agree on the timing.  The job time is the slowest
rank's device time and the job throughput is the work of all ranks over that time.
"""
from __future__ import annotations

import os


def dist_env():
    """(rank, local_rank, world_size) from the launcher's environment."""
    return (int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)),
            int(os.environ.get("WORLD_SIZE", 1)))


def replica_seed(base_seed: int, rank: int) -> int:
    """Every replica fills its cache from its own random stream."""
    return base_seed + 1000 * rank


def max_over_ranks(values, device=None):
    """Element-wise maximum of a list of floats over all ranks (identity for a single process)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def job_throughput_gbs(bytes_per_call: int, calls_per_rank: int, world: int, slowest_ms: float) -> float:
    """Aggregate K/V GB/s of the whole job: all ranks' bytes over the slowest rank's time."""
    return bytes_per_call * calls_per_rank * world / (slowest_ms * 1e-3) / 1e9


def sharded_throughput_gbs(whole_cache_bytes: int, calls: int, slowest_ms: float) -> float:
    """K/V GB/s of a key-range-sharded job: the whole cache is streamed once per layer call, each rank
    reading its own share, and a call is over when the slowest rank has merged the gathered partials."""
    return whole_cache_bytes * calls / (slowest_ms * 1e-3) / 1e9
