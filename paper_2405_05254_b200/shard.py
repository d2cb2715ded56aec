"""Host-side plumbing for key-range sharding of one long K/V cache across GPUs.

Each rank keeps a contiguous range of every sequence's keys (the state sequence-parallel prefill
leaves behind), runs ``yoco_xattn_decode_partial`` on what it holds, and the ranks exchange their
``[rows, d]`` partial rows and ``[rows]`` log-sum-exps (about 16 KB per layer call at T = 1) before
each merges them locally with ``yoco_xattn_combine_gathered``.  The merge is algebraically exact,
so the sharded result is the unsharded one up to rounding order.

Nothing here computes attention: it cuts index ranges, slices packed buffers and moves tensors.
"""
from __future__ import annotations

import numpy as np


def key_range_shards(kv_len, world: int, tile: int = 64):
    """Contiguous key ranges per rank: returns (offset[world, B], count[world, B]) int32.

    Every range but a sequence's last starts and ends on a multiple of ``tile`` keys (the decode
    kernel's tile), ranges are as even as that allows, and short sequences leave the last ranks
    empty.  The ranges of one sequence partition [0, N) exactly."""
    kv_len = np.asarray(kv_len, dtype=np.int64)
    if world <= 0 or tile <= 0 or (kv_len < 0).any():
        raise ValueError("world and tile must be positive, lengths non-negative")
    tiles = -(-kv_len // tile)
    per_rank = -(-tiles // world) * tile                      # keys per rank, tile-aligned
    r = np.arange(world, dtype=np.int64).reshape(-1, 1)
    lo = np.minimum(r * per_rank, kv_len)
    hi = np.minimum((r + 1) * per_rank, kv_len)
    return lo.astype(np.int32), (hi - lo).astype(np.int32)


def take_key_range(packed: np.ndarray, kv_len, Hkv: int, d: int, offset, count) -> np.ndarray:
    """Cuts keys [offset[i], offset[i] + count[i]) of every sequence and KV head out of a tightly
    packed cache ([Hkv, N_i, d] per sequence, sequences back to back) and packs them the same way."""
    packed = np.asarray(packed).reshape(-1)
    out = np.empty(int(np.sum(count)) * Hkv * d, dtype=packed.dtype)
    src = dst = 0
    for n, o, c in zip(np.asarray(kv_len, dtype=np.int64), offset, count):
        seq = packed[src:src + Hkv * n * d].reshape(Hkv, n, d)
        out[dst:dst + Hkv * c * d] = seq[:, o:o + c].reshape(-1)
        src += Hkv * n * d
        dst += Hkv * int(c) * d
    return out


def exchange_partials(part_o, part_lse, group=None):
    """All-gather of every rank's partial rows: ([rows, d], [rows]) -> ([S, rows, d], [S, rows]) with
    S = world size, rank-major -- the layout ``yoco_xattn_combine_gathered`` reads.  A single process
    (no process group) just gets a leading axis of one."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return part_o.unsqueeze(0).contiguous(), part_lse.unsqueeze(0).contiguous()
    S = dist.get_world_size(group)
    all_o = torch.empty((S,) + tuple(part_o.shape), dtype=part_o.dtype, device=part_o.device)
    all_l = torch.empty((S,) + tuple(part_lse.shape), dtype=part_lse.dtype, device=part_lse.device)
    # output as the concatenation along the first axis (the form every backend accepts)
    dist.all_gather_into_tensor(all_o.view(-1, *part_o.shape[1:]), part_o.contiguous(), group=group)
    dist.all_gather_into_tensor(all_l.view(-1, *part_lse.shape[1:]), part_lse.contiguous(), group=group)
    return all_o, all_l
