"""Parity of the split-KV decode path (through the C ABI) against the fp64 oracle."""
import math

import numpy as np
import pytest

import oracle
import synth_inputs as si
from helpers import GpuRunner, assert_close, assert_lse_close, bf16_dev_to_f64, errors, to_dev_bf16

pytestmark = pytest.mark.gpu


def oracle_full(w, Q, K, V, **kw):
    return oracle.xattn(Q, K, V, w.cu, w.kv_len, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=w.T, **kw)


def run_workload(w, layers=None, mode="decode"):
    K, V = w.make_k(), w.make_v()
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, w.T, w.kv_len, K, V)
    out = []
    for l in range(w.layers if layers is None else layers):
        Q = w.make_q(l)
        o, lse, _ = r.run(Q, mode)
        o_ref, lse_ref = oracle_full(w, Q, K, V)
        out.append(assert_close(o, o_ref, f"{w.name} layer {l}"))
        assert_lse_close(lse, lse_ref, f"{w.name} layer {l}")
    return out


def test_tiny_config_two_layers_share_one_cache():
    run_workload(si.workload("tiny"))


def test_3b_class_32k_all_thirteen_layers():
    run_workload(si.workload("3b_32k"))


def test_ragged_small_batch():
    run_workload(si.workload("ragged_small"))


@pytest.mark.parametrize("N", [1, 2, 15, 16, 17, 63, 64, 65, 127, 129, 1000, 4097])
def test_lengths_around_tile_edges(N):
    w = si.Workload("edge", B=2, Hq=8, Hkv=2, d=128, T=1, layers=1, seed=100 + N, kv_len=[N, max(1, N // 2)])
    run_workload(w)


@pytest.mark.parametrize("Hq,Hkv,T,d", [(24, 8, 1, 128), (8, 8, 1, 128), (32, 8, 2, 128), (32, 8, 4, 128),
                                        (16, 1, 1, 128), (6, 2, 5, 64), (4, 4, 16, 64), (8, 2, 3, 128)])
def test_group_sizes_and_small_chunks(Hq, Hkv, T, d):
    """G = 3 (the paper's 24/8 heads), MHA, and T > 1 rows that are causal among themselves."""
    w = si.Workload("grp", B=3, Hq=Hq, Hkv=Hkv, d=d, T=T, layers=1, seed=7, kv_len=[700, 64 + T, 333])
    run_workload(w)


def test_more_query_rows_than_keys_and_empty_sequences():
    w = si.Workload("short", B=4, Hq=8, Hkv=2, d=128, T=4, layers=1, seed=8, kv_len=[2, 0, 4, 1])
    K, V = w.make_k(), w.make_v()
    Q = w.make_q(0)
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, w.T, w.kv_len, K, V)
    o, lse, _ = r.run(Q)
    o_ref, lse_ref = oracle_full(w, Q, K, V)
    assert_close(o, o_ref, "short")
    assert_lse_close(lse, lse_ref, "short")
    assert (o[1] == 0).all() and np.isneginf(lse[1]).all()        # empty sequence
    assert (o[0, :, :2] == 0).all()                                # rows with no visible key


def test_peaked_scores_exercise_the_rescale_path():
    """A few keys late in the sequence with much larger scores force the running max to move."""
    w = si.Workload("peaked", B=1, Hq=32, Hkv=8, d=128, T=1, layers=1, seed=9, kv_len=[20000])
    K, V = w.make_k().reshape(8, 20000, 128).copy(), w.make_v()
    Q = w.make_q(0)
    qf = si.bf16_bits_to_f32(Q).reshape(8, 4, 128)
    for c in range(8):
        for n, (pos, gain) in enumerate([(5000, 0.4), (12345, 0.8), (19990, 1.2), (19999, 1.0)]):
            K[c, pos] = si.f32_to_bf16_bits(gain * qf[c, n % 4])
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, w.T, w.kv_len, K, V)
    o, lse, _ = r.run(Q)
    o_ref, lse_ref = oracle_full(w, Q, K.reshape(-1), V)
    assert_close(o, o_ref, "peaked")
    assert_lse_close(lse, lse_ref, "peaked")
    assert np.abs(o_ref).max() > 0.5      # the peaks really dominate some heads


def test_one_hot_selection_is_bit_exact_at_every_split_and_tile_edge():
    """One key leads by > 150 in the exponent, so every other weight is exactly 0 in fp32 and the
    output must equal that key's V bit for bit, wherever the key sits: first/last key of each
    split, of each 64-key tile, of each warp's 16-key slice and of each ragged sequence."""
    from paper_2405_05254_b200 import binding as bd
    B, Hq, Hkv, d = 3, 8, 2, 128
    lens = np.array([5000, 777, 64], dtype=np.int32)
    w = si.Workload("onehot", B=B, Hq=Hq, Hkv=Hkv, d=d, T=1, layers=1, seed=10, kv_len=lens)
    V = w.make_v()
    shape = bd.make_shape(B, Hq, Hkv, d, 1)
    _, segs = bd.yoco_xattn_plan(shape, lens, 148, bd.MODE_DECODE)
    positions = {b: set() for b in range(B)}
    for s in segs:
        positions[s.b] |= {s.k_begin, s.k_end - 1}
    for b in range(B):
        n = int(lens[b])
        positions[b] |= {0, n - 1, 15, 16, 63, 64} & set(range(n))
    Q = si.f32_to_bf16_bits(np.full((B, Hq, 1, d), 16.0, dtype=np.float32))
    Vf = si.bf16_bits_to_f32(V)
    r = None
    rounds = max(len(p) for p in positions.values())
    for k in range(rounds):
        K = np.zeros(w.kv_elems, dtype=np.float32)
        picks = []
        for b in range(B):
            plist = sorted(positions[b])
            j = plist[k % len(plist)]
            picks.append(j)
            for c in range(Hkv):
                base = int(w.cu[b]) * Hkv * d + (c * int(lens[b]) + j) * d
                K[base:base + d] = 8.0
        r = GpuRunner(B, Hq, Hkv, d, 1, lens, si.f32_to_bf16_bits(K), V)
        o, lse, _ = r.run(Q)
        for b in range(B):
            for h in range(Hq):
                c = h // (Hq // Hkv)
                base = int(w.cu[b]) * Hkv * d + (c * int(lens[b]) + picks[b]) * d
                np.testing.assert_array_equal(o[b, h, 0], Vf[base:base + d].astype(np.float64),
                                              err_msg=f"b={b} h={h} key={picks[b]}")
        assert np.allclose(lse, 16 * 8 * d / math.sqrt(d), rtol=1e-6)


def test_cache_with_spare_capacity_per_head_and_garbage_beyond_the_length():
    """kv_head_stride > N*d; the slack rows hold NaN bit patterns and must not leak into O."""
    B, Hq, Hkv, d, cap = 2, 8, 2, 128, 300
    lens = np.array([257, 100], dtype=np.int32)
    rng = np.random.default_rng(3)
    K = np.full((B, Hkv, cap, d), 0x7FC0, dtype=np.uint16)    # NaN everywhere
    V = np.full((B, Hkv, cap, d), 0x7FC0, dtype=np.uint16)
    for b in range(B):
        n = int(lens[b])
        K[b, :, :n] = si.f32_to_bf16_bits(rng.standard_normal((Hkv, n, d)).astype(np.float32))
        V[b, :, :n] = si.f32_to_bf16_bits(rng.standard_normal((Hkv, n, d)).astype(np.float32))
    Q = si.f32_to_bf16_bits(rng.standard_normal((B, Hq, 1, d)).astype(np.float32))
    cu = np.array([0, cap, 2 * cap], dtype=np.int32)
    r = GpuRunner(B, Hq, Hkv, d, 1, lens, K, V, cu=cu, kv_head_stride=cap * d)
    o, lse, _ = r.run(Q)
    o_ref, lse_ref = oracle.xattn(Q, K, V, cu, lens, B=B, Hq=Hq, Hkv=Hkv, d=d, T=1, kv_head_stride=cap * d)
    assert_close(o, o_ref, "capacity layout")
    assert_lse_close(lse, lse_ref, "capacity layout")


def test_explicit_scale_and_no_lse_output():
    w = si.Workload("scale", B=1, Hq=8, Hkv=2, d=64, T=1, layers=1, seed=11, kv_len=[900])
    K, V, Q = w.make_k(), w.make_v(), w.make_q(0)
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, w.T, w.kv_len, K, V, scale=0.31)
    o, _, _ = r.run(Q, want_lse=False)
    o_ref, _ = oracle_full(w, Q, K, V, scale=0.31)
    assert_close(o, o_ref, "explicit scale")


def test_two_runs_are_bit_identical():
    import torch
    w = si.workload("ragged_small")
    K, V, Q = w.make_k(), w.make_v(), w.make_q(0)
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, w.T, w.kv_len, K, V)
    _, _, O1 = r.run(Q)
    a = O1.clone()
    _, _, O2 = r.run(Q)
    assert torch.equal(a.view(torch.int16), O2.view(torch.int16))


def test_combine_entry_point_against_the_oracle():
    import torch
    from paper_2405_05254_b200 import binding as bd
    rng = np.random.default_rng(12)
    for rows, S, d in [(37, 5, 128), (4, 1, 64), (130, 40, 128), (3, 33, 256)]:
        po = rng.standard_normal((rows, S, d)).astype(np.float32)
        pl = (4 * rng.standard_normal((rows, S))).astype(np.float32)
        pl[rng.random((rows, S)) < 0.2] = -np.inf
        pl[0, :] = -np.inf
        O = torch.empty((rows, d), dtype=torch.bfloat16, device="cuda")
        L = torch.empty((rows,), dtype=torch.float32, device="cuda")
        bd.yoco_xattn_combine(torch.from_numpy(po).cuda(), torch.from_numpy(pl).cuda(), O, L)
        torch.cuda.synchronize()
        o_ref, l_ref = oracle.combine(po, pl)
        from helpers import bf16_dev_to_f64
        assert_close(bf16_dev_to_f64(O).reshape(rows, d), o_ref, f"combine {rows}x{S}x{d}")
        assert_lse_close(L.cpu().numpy(), l_ref, "combine lse")


def test_combine_with_one_live_piece_is_a_bit_exact_pass_through():
    import torch
    from paper_2405_05254_b200 import binding as bd
    rng = np.random.default_rng(13)
    rows, S, d = 16, 7, 128
    po = rng.standard_normal((rows, S, d)).astype(np.float32)
    pl = np.full((rows, S), -np.inf, dtype=np.float32)
    live = rng.integers(0, S, size=rows)
    pl[np.arange(rows), live] = rng.standard_normal(rows).astype(np.float32) * 10
    O = torch.empty((rows, d), dtype=torch.bfloat16, device="cuda")
    bd.yoco_xattn_combine(torch.from_numpy(po).cuda(), torch.from_numpy(pl).cuda(), O)
    want = torch.from_numpy(po[np.arange(rows), live]).bfloat16()
    assert torch.equal(O.cpu().view(torch.int16), want.view(torch.int16))


def test_undersized_workspace_is_refused():
    import torch
    from paper_2405_05254_b200 import binding as bd
    shape = bd.make_shape(1, 32, 8, 128, 1, max_kv_len=4096)
    t = torch.zeros(4096 * 8 * 128, dtype=torch.bfloat16, device="cuda")
    q = torch.zeros(32 * 128, dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(512, dtype=torch.uint8, device="cuda")
    with pytest.raises(bd.YocoError) as e:
        bd.yoco_xattn_decode(shape, q, t, t, None, [4096], q.clone(), None, ws)
    assert e.value.code == bd.ERR_WORKSPACE_TOO_SMALL


@pytest.mark.parametrize("lens", [[20000, 333], [250000, 333]])
def test_layer_calls_replay_bit_identically_from_a_cuda_graph(lens):
    """A serving loop captures the layer calls of a step once and replays them: the call only
    enqueues (header memset, attention kernel, merge), so a capture on a side stream must replay
    to the same bits as the eager calls -- also when the groups run in pieces handed out at run time
    (the long case), whose work counter is reset by the captured memset at every replay."""
    import torch
    from paper_2405_05254_b200 import binding as bd
    w = si.Workload("graph", B=2, Hq=32, Hkv=8, d=128, T=1, layers=3, seed=29, kv_len=lens)
    K, V = to_dev_bf16(w.make_k()), to_dev_bf16(w.make_v())
    Qs = [to_dev_bf16(w.make_q(l).reshape(-1)) for l in range(w.layers)]
    Os = [torch.empty(w.B * w.Hq * w.d, dtype=torch.bfloat16, device="cuda") for _ in range(w.layers)]
    shape = bd.make_shape(w.B, w.Hq, w.Hkv, w.d, 1, max_kv_len=int(w.kv_len.max()))
    ws = torch.empty(bd.yoco_xattn_workspace_size(shape, w.kv_len, bd.MODE_DECODE), dtype=torch.uint8, device="cuda")
    side = torch.cuda.Stream()

    def step():
        for l in range(w.layers):
            bd.yoco_xattn_decode(shape, Qs[l], K, V, w.cu, w.kv_len, Os[l], None, ws, side)

    with torch.cuda.stream(side):
        step()                                   # first call outside the capture: one-time set-up
    torch.cuda.synchronize()
    eager = [o.clone() for o in Os]
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        step()
    for _ in range(3):
        for o in Os:
            o.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert bd.yoco_xattn_status(ws, side) == 0
        for a, b in zip(eager, Os):
            assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_a_recorded_call_with_tables_in_the_workspace_survives_plan_cache_eviction():
    """A problem too large for kernel-parameter tables uploads them from the library's plan cache.  Recorded
    into a graph, that copy reads the plan's host memory again at every replay, so the library keeps such a
    plan for good: after enough other shapes to push it out of the 16-entry cache the replay must still give
    the oracle's result.  (Where the CUDA runtime refuses to record a copy from pageable memory the call must
    fail with an error code and leave the context usable.)"""
    import torch
    from paper_2405_05254_b200 import binding as bd
    w = si.Workload("graph_big", B=25, Hq=8, Hkv=8, d=128, T=1, layers=1, seed=30,
                    kv_len=[4000 + 137 * i for i in range(25)])          # 200 streams, ~490 segments
    Kb, Vb, Qb = w.make_k(), w.make_v(), w.make_q(0)
    K, V, Q = to_dev_bf16(Kb), to_dev_bf16(Vb), to_dev_bf16(Qb.reshape(-1))
    O = torch.empty(w.B * w.Hq * w.d, dtype=torch.bfloat16, device="cuda")
    shape = bd.make_shape(w.B, w.Hq, w.Hkv, w.d, 1, max_kv_len=int(w.kv_len.max()))
    ws = torch.empty(bd.yoco_xattn_workspace_size(shape, w.kv_len, bd.MODE_DECODE), dtype=torch.uint8, device="cuda")
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        bd.yoco_xattn_decode(shape, Q, K, V, w.cu, w.kv_len, O, None, ws, side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    try:
        with torch.cuda.graph(graph, stream=side):
            bd.yoco_xattn_decode(shape, Q, K, V, w.cu, w.kv_len, O, None, ws, side)
    except (bd.YocoError, RuntimeError) as e:
        torch.cuda.synchronize()
        assert int(torch.zeros(1, device="cuda").item()) == 0          # refused cleanly, context alive
        pytest.skip(f"the runtime does not record this copy: {e}")
    # 20 other shapes through the same entry point: the recorded plan leaves the cache
    small = torch.zeros(64 * 8 * 128, dtype=torch.bfloat16, device="cuda")
    for n in range(1, 21):
        sh = bd.make_shape(1, 8, 8, 128, 1, max_kv_len=n)
        wsn = torch.empty(bd.yoco_xattn_workspace_size(sh, [n], bd.MODE_DECODE), dtype=torch.uint8, device="cuda")
        bd.yoco_xattn_decode(sh, small, small, small, None, [n], small.clone(), None, wsn)
    torch.cuda.synchronize()
    o_ref, _ = oracle_full(w, Qb, Kb, Vb)
    for _ in range(2):
        O.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert bd.yoco_xattn_status(ws, side) == 0
        assert_close(bf16_dev_to_f64(O).reshape(o_ref.shape), o_ref, "replay after eviction")


def test_calls_on_two_streams_with_their_own_workspaces_do_not_interfere():
    """Two serving streams, different problems, interleaved calls: each has its own workspace, the
    plan cache and the launches must keep them apart."""
    import torch
    from paper_2405_05254_b200 import binding as bd
    ws_list, outs, refs, streams = [], [], [], [torch.cuda.Stream(), torch.cuda.Stream()]
    probs = [si.Workload("s0", B=1, Hq=32, Hkv=8, d=128, T=1, layers=2, seed=71, kv_len=[30000]),
             si.Workload("s1", B=3, Hq=8, Hkv=2, d=64, T=2, layers=2, seed=72, kv_len=[5000, 77, 1300])]
    state = []
    for w in probs:
        K, V = to_dev_bf16(w.make_k()), to_dev_bf16(w.make_v())
        Qs = [to_dev_bf16(w.make_q(l).reshape(-1)) for l in range(w.layers)]
        Os = [torch.empty(w.B * w.Hq * w.T * w.d, dtype=torch.bfloat16, device="cuda") for _ in range(w.layers)]
        shape = bd.make_shape(w.B, w.Hq, w.Hkv, w.d, w.T, max_kv_len=int(w.kv_len.max()))
        ws = torch.empty(bd.yoco_xattn_workspace_size(shape, w.kv_len, bd.MODE_DECODE), dtype=torch.uint8, device="cuda")
        state.append((w, K, V, Qs, Os, shape, ws))
    torch.cuda.synchronize()
    for rep in range(3):
        for l in range(2):
            for (w, K, V, Qs, Os, shape, ws), st in zip(state, streams):
                bd.yoco_xattn_decode(shape, Qs[l], K, V, w.cu, w.kv_len, Os[l], None, ws, st)
    torch.cuda.synchronize()
    for (w, K, V, Qs, Os, shape, ws), st in zip(state, streams):
        assert bd.yoco_xattn_status(ws, st) == 0
        for l in range(2):
            o_ref, _ = oracle.xattn(w.make_q(l), w.make_k(), w.make_v(), w.cu, w.kv_len, B=w.B, Hq=w.Hq, Hkv=w.Hkv,
                                    d=w.d, T=w.T)
            got = si.bf16_bits_to_f32(Os[l].view(torch.int16).cpu().numpy().view(np.uint16)).astype(np.float64)
            assert_close(got.reshape(o_ref.shape), o_ref, f"{w.name} layer {l}")


def test_long_ragged_batch_runs_its_groups_in_pieces():
    """Sequences long enough for the plan to cut every group into pieces, with lengths chosen so
    that groups straddle stream boundaries (a piece then holds nothing of one of its group's
    segments and must mark that slot empty).  All rows against the oracle, and the plan says what ran."""
    import torch
    from paper_2405_05254_b200 import binding as bd
    lens = np.array([200001, 130000, 70003], dtype=np.int32)
    w = si.Workload("pieces", B=3, Hq=8, Hkv=2, d=128, T=1, layers=1, seed=21, kv_len=lens)
    sm = torch.cuda.get_device_properties(0).multi_processor_count
    info, segs = bd.yoco_xattn_plan(bd.make_shape(w.B, w.Hq, w.Hkv, w.d, 1), lens, sm, bd.MODE_DECODE)
    assert info.sub_items == 2 or info.sub_items == 4
    assert info.num_segments < info.num_slots          # some piece is empty for some segment
    K, V, Q = w.make_k(), w.make_v(), w.make_q(0)
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, 1, lens, K, V)
    o, lse, _ = r.run(Q)
    o_ref, lse_ref = oracle.xattn(Q, K, V, w.cu, lens, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=1)
    assert_close(o, o_ref, "pieces")
    assert_lse_close(lse, lse_ref, "pieces")


def test_pieces_give_the_same_bits_whoever_runs_them():
    """Which CTA runs a piece depends on timing; the result must not.  The same call repeated, alone
    and while another stream keeps the SMs busy with a second problem, is bit-identical every time."""
    import torch
    from paper_2405_05254_b200 import binding as bd
    w = si.Workload("pieces2", B=1, Hq=32, Hkv=8, d=128, T=1, layers=1, seed=22, kv_len=[300000])
    K, V, Q = w.make_k(), w.make_v(), w.make_q(0)
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, 1, w.kv_len, K, V)
    sm = torch.cuda.get_device_properties(0).multi_processor_count
    info, _ = bd.yoco_xattn_plan(r.shape, w.kv_len, sm, bd.MODE_DECODE)
    assert info.sub_items == 4
    o0, lse0, O = r.run(Q)
    ref_bits, ref_lse = O.view(torch.int16).clone(), lse0.copy()
    o_ref, lse_ref = oracle.xattn(Q, K, V, w.cu, w.kv_len, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=1)
    assert_close(o0, o_ref, "four pieces")
    assert_lse_close(lse0, lse_ref, "four pieces")
    # a second, smaller problem on another stream perturbs who is free when
    w2 = si.Workload("noise", B=4, Hq=8, Hkv=8, d=128, T=1, layers=1, seed=23, kv_len=[9000, 14000, 300, 7000])
    r2 = GpuRunner(w2.B, w2.Hq, w2.Hkv, w2.d, 1, w2.kv_len, w2.make_k(), w2.make_v())
    O2, L2, W2 = r2._buffers(bd.MODE_DECODE)
    Q2 = to_dev_bf16(w2.make_q(0).reshape(-1))
    side = torch.cuda.Stream()
    for rep in range(6):
        if rep >= 2:
            with torch.cuda.stream(side):
                for _ in range(8):
                    bd.yoco_xattn_decode(r2.shape, Q2, r2.K, r2.V, None, w2.kv_len, O2, L2, W2, stream=side)
        o, lse, O = r.run(Q)
        assert torch.equal(O.view(torch.int16), ref_bits), f"repeat {rep} differs"
        assert np.array_equal(lse, ref_lse)
    torch.cuda.synchronize()
    assert bd.yoco_xattn_status(W2) == 0


def test_prepared_call_gives_the_same_bits_as_the_plain_call():
    import torch
    from paper_2405_05254_b200 import binding as bd
    w = si.workload("ragged_small")
    r = GpuRunner(w.B, w.Hq, w.Hkv, w.d, w.T, w.kv_len, w.make_k(), w.make_v())
    _, _, O1 = r.run(w.make_q(0))
    want = O1.view(torch.int16).clone()
    O, L, W = r._buffers(bd.MODE_DECODE)
    Q = to_dev_bf16(w.make_q(0).reshape(-1))
    call = bd.prepare_decode(r.shape, Q, r.K, r.V, r.cu, r.kv_len, O, L, W)
    for _ in range(3):
        O.zero_()
        call.run()
        assert bd.yoco_xattn_status(W) == 0
        assert torch.equal(O.view(torch.int16), want)
