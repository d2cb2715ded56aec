"""Parity of the sliding-window mask (Section 3.2: row i sees i - C < j <= i) on the CUDA path,
through the C ABI, against the fp64 oracle: decode kernel and both chunk kernels."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from helpers import GpuRunner, assert_close, assert_lse_close

pytestmark = pytest.mark.gpu


def run(w, mode, C):
    K, V, Q = w.make_k(), w.make_v(), w.make_q(0)
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, w.T, w.kv_len, K, V, window=C)
    o, lse, _ = r.run(Q, mode)
    o_ref, lse_ref = oracle.xattn(Q, K, V, w.cu, w.kv_len, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=w.T, window=C)
    assert_close(o, o_ref, f"{w.name} {mode} C={C}")
    assert_lse_close(lse, lse_ref, f"{w.name} {mode} C={C}")
    return o, K, V


@pytest.mark.parametrize("C", [1, 63, 64, 65, 100, 1000, 10 ** 6])
def test_decode_window_on_a_ragged_batch(C):
    run(si.Workload("win_dec", B=4, Hq=32, Hkv=8, d=128, T=1, layers=1, seed=50, kv_len=[700, 64, 3000, 1]),
        "decode", C)


@pytest.mark.parametrize("C", [2, 200])
def test_decode_window_with_several_rows_per_head(C):
    run(si.Workload("win_dec_t", B=2, Hq=8, Hkv=2, d=64, T=4, layers=1, seed=51, kv_len=[500, 5]), "decode", C)


def test_decode_window_far_into_a_long_cache_reads_only_the_window():
    """N = 40,000 with C = 1,024: the plan starts at the window, the result is the oracle's."""
    w = si.Workload("win_long", B=1, Hq=32, Hkv=8, d=128, T=1, layers=1, seed=52, kv_len=[40000])
    run(w, "decode", 1024)
    from paper_2405_05254_b200 import binding as bd
    info, segs = bd.yoco_xattn_plan(bd.make_shape(1, 32, 8, 128, 1, window=1024), w.kv_len, 148, bd.MODE_DECODE)
    assert info.total_tiles == 8 * 16 and min(s.k_begin for s in segs) == 38976


@pytest.mark.parametrize("C", [1, 50, 128, 129, 700, 5000])
@pytest.mark.parametrize("shape", ["one_tile", "pair"])
def test_chunk_window(shape, C):
    if shape == "one_tile":      # 128 rows per stream: the one-tile kernel
        w = si.Workload("win_chunk1", B=2, Hq=4, Hkv=1, d=128, T=32, layers=1, seed=53, kv_len=[1000, 33])
    else:                        # 640 rows per stream: the two-tile kernel
        w = si.Workload("win_chunk2", B=2, Hq=32, Hkv=8, d=128, T=160, layers=1, seed=54, kv_len=[1160, 937])
    run(w, "chunk", C)


@pytest.mark.parametrize("mode,T", [("decode", 1), ("decode", 3), ("chunk", 3), ("chunk", 200)])
def test_window_of_one_is_bit_exact(mode, T):
    """C = 1 keeps the row's own key only: weight exactly 1, so O must be V[i] bit for bit."""
    w = si.Workload("win_one", B=1, Hq=4, Hkv=1, d=128, T=T, layers=1, seed=55, kv_len=[777])
    o, K, V = run(w, mode, 1)
    Vf = si.bf16_bits_to_f32(V).reshape(777, 128).astype(np.float64)
    for t in range(T):
        for h in range(4):
            np.testing.assert_array_equal(o[0, h, t], Vf[777 - T + t])
