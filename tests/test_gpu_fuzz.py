"""Seeded random shapes through every attention entry point against the oracle: ragged lengths, odd
group sizes, windows, caches with spare capacity, lengths around tile and split boundaries."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from helpers import GpuRunner, assert_close, assert_lse_close

pytestmark = pytest.mark.gpu


def random_case(rng, mode):
    d = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 3, 8]))
    if mode == "decode":
        G = int(rng.choice([1, 2, 3, 4, 8, 16]))
        T = int(rng.integers(1, 16 // G + 1))
    else:
        G = int(rng.choice([1, 3, 4, 8]))
        T = int(rng.choice([1, 7, 32, 33, 100, 129, 260]))
    B = int(rng.integers(1, 5))
    edges = [1, 63, 64, 65, 127, 128, 129, 191, 192, 1000, 2049, 5000, 9000]
    lens = [int(rng.choice(edges)) + int(rng.integers(0, 3)) for _ in range(B)]
    if rng.random() < 0.3:
        lens[int(rng.integers(0, B))] = 0
    window = int(rng.choice([0, 0, 1, 50, 64, 200, 4096]))
    cap = int(rng.choice([0, 0, 1])) * (max(lens) + int(rng.integers(0, 70)))
    return dict(B=B, Hq=G * Hkv, Hkv=Hkv, d=d, T=T, lens=lens, window=window, cap=cap)


@pytest.mark.parametrize("mode", ["decode", "chunk"])
@pytest.mark.parametrize("seed", range(12))
def test_random_shapes(mode, seed):
    rng = np.random.default_rng(1000 * (mode == "chunk") + seed)
    c = random_case(rng, mode)
    B, Hq, Hkv, d, T, lens, cap = c["B"], c["Hq"], c["Hkv"], c["d"], c["T"], np.array(c["lens"], np.int32), c["cap"]
    Q = si.f32_to_bf16_bits(rng.standard_normal((B, Hq, T, d)).astype(np.float32))
    if cap:     # spare rows per head, filled with NaN bit patterns
        K = np.full((B, Hkv, cap, d), 0x7FC0, dtype=np.uint16)
        V = np.full((B, Hkv, cap, d), 0x7FC0, dtype=np.uint16)
        for i, n in enumerate(lens):
            K[i, :, :n] = si.f32_to_bf16_bits(rng.standard_normal((Hkv, n, d)).astype(np.float32))
            V[i, :, :n] = si.f32_to_bf16_bits(rng.standard_normal((Hkv, n, d)).astype(np.float32))
        cu, stride = (np.arange(B + 1) * cap).astype(np.int32), cap * d
    else:
        tot = int(lens.sum()) * Hkv * d
        K = si.f32_to_bf16_bits(rng.standard_normal(max(tot, 8)).astype(np.float32))
        V = si.f32_to_bf16_bits(rng.standard_normal(max(tot, 8)).astype(np.float32))
        cu, stride = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32), 0
    r = GpuRunner(B, Hq, Hkv, d, T, lens, K, V, cu=cu if cap else None, kv_head_stride=stride, window=c["window"])
    o, lse, _ = r.run(Q, mode)
    o_ref, lse_ref = oracle.xattn(Q, K, V, cu, lens, B=B, Hq=Hq, Hkv=Hkv, d=d, T=T, kv_head_stride=stride,
                                  window=c["window"])
    assert_close(o, o_ref, str(c))
    assert_lse_close(lse, lse_ref, str(c))


def random_long_case(rng):
    """Caches long enough for the decode plan to cut its groups into pieces (40 key tiles or more per group
    on 148 SMs: about 760,000 keys over all streams), few streams, every option of the call."""
    d = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 4, 8]))
    G = int(rng.choice([1, 2, 4, 8, 16]))
    T = int(rng.integers(1, 16 // G + 1))
    B = int(rng.integers(1, 4))
    total = int(rng.integers(800_000, 2_400_000)) // Hkv          # keys per head, all sequences together
    cuts = np.sort(rng.integers(1, total, size=B - 1)) if B > 1 else np.array([], dtype=np.int64)
    lens = np.diff(np.concatenate([[0], cuts, [total]])).astype(np.int64)
    lens = [int(max(n, T)) + int(rng.integers(0, 3)) for n in lens]
    window = int(rng.choice([0, 0, 0, 300_000, 65]))
    cap = int(rng.choice([0, 0, 1])) * (max(lens) + int(rng.integers(0, 70)))
    return dict(B=B, Hq=G * Hkv, Hkv=Hkv, d=d, T=T, lens=lens, window=window, cap=cap)


@pytest.mark.parametrize("seed", range(6))
def test_random_long_caches_in_pieces(seed):
    import torch
    from paper_2405_05254_b200 import binding as bd
    rng = np.random.default_rng(5000 + seed)
    c = random_long_case(rng)
    B, Hq, Hkv, d, T, lens, cap = c["B"], c["Hq"], c["Hkv"], c["d"], c["T"], np.array(c["lens"], np.int32), c["cap"]
    gen = lambda *shape: si.f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32))      # noqa: E731
    Q = gen(B, Hq, T, d)
    if cap:
        K = np.full((B, Hkv, cap, d), 0x7FC0, dtype=np.uint16)
        V = np.full((B, Hkv, cap, d), 0x7FC0, dtype=np.uint16)
        for i, n in enumerate(lens):
            K[i, :, :n] = gen(Hkv, int(n), d)
            V[i, :, :n] = gen(Hkv, int(n), d)
        cu, stride = (np.arange(B + 1) * cap).astype(np.int32), cap * d
    else:
        tot = int(lens.sum()) * Hkv * d
        K, V = gen(tot), gen(tot)
        cu, stride = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32), 0
    r = GpuRunner(B, Hq, Hkv, d, T, lens, K, V, cu=cu if cap else None, kv_head_stride=stride, window=c["window"])
    sm = torch.cuda.get_device_properties(0).multi_processor_count
    info, _ = bd.yoco_xattn_plan(r.shape, lens, sm, bd.MODE_DECODE)
    o, lse, _ = r.run(Q, "decode")
    o_ref, lse_ref = oracle.xattn(Q, K, V, cu, lens, B=B, Hq=Hq, Hkv=Hkv, d=d, T=T, kv_head_stride=stride,
                                  window=c["window"])
    assert_close(o, o_ref, f"{c} pieces={info.sub_items}")
    assert_lse_close(lse, lse_ref, f"{c} pieces={info.sub_items}")
