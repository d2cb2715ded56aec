"""Host-side checks (no GPU): the library loads, exports the declared symbols, validates
arguments before touching CUDA, and the split/tile planner partitions the key space exactly."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2405_05254_b200 import binding as bd

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            src = open(os.path.join(ROOT, "include", fn)).read()
            names |= set(re.findall(r"\b(yoco_(?:xattn|kv)_[a-z_0-9]+)\s*\(", src))
    return sorted(names)


def test_library_exports_every_declared_symbol():
    L = bd.lib()
    syms = declared_symbols()
    assert {"yoco_xattn_decode", "yoco_xattn_chunk", "yoco_xattn_combine", "yoco_xattn_plan",
            "yoco_xattn_workspace_size", "yoco_xattn_status", "yoco_xattn_strerror", "yoco_xattn_decode_partial",
            "yoco_xattn_combine_gathered", "yoco_xattn_decode_fp8", "yoco_kv_append", "yoco_kv_fold_gain",
            "yoco_kv_append_status", "yoco_kv_append_fp8"} <= set(syms)
    for s in syms:
        assert hasattr(L, s), f"{s} is declared in include/ but not exported"


def test_strerror_covers_the_codes():
    msgs = {bd.lib().yoco_xattn_strerror(c) for c in range(-5, 1)}
    assert len(msgs) == 6 and b"unknown error code" not in msgs
    assert bd.lib().yoco_xattn_strerror(-99) == b"unknown error code"


def restated_plan(B, Hkv, lens, sm_count, mode, G, T):
    """Test-side restatement of the rule: flat (stream, tile) space cut into equal ranges."""
    tile_n = 64 if mode == bd.MODE_DECODE else 128
    tile_m = 16 if mode == bd.MODE_DECODE else (256 if G * T > 128 else 128)
    m_tiles = -(-G * T // tile_m)
    nts = [-(-int(n) // tile_n) for n in lens]
    total = Hkv * sum(nts)
    target = sm_count * 2 if mode == bd.MODE_DECODE else max(1, sm_count // m_tiles)
    groups = max(1, min(target, total))
    bounds = [p * total // groups for p in range(groups + 1)]
    segs = []
    flat = 0
    for b in range(B):
        for c in range(Hkv):
            lo, hi = flat, flat + nts[b]
            for p in range(groups):
                a, e = max(lo, bounds[p]), min(hi, bounds[p + 1])
                if a < e:
                    segs.append((p, b, c, (a - lo) * tile_n, min((e - lo) * tile_n, int(lens[b]))))
            flat = hi
    # decode groups of 40 tiles or more are cut once more, into 2 or 4 pieces of decreasing size
    R = 1
    if mode == bd.MODE_DECODE:
        per = total // groups
        R = 4 if per >= 96 else 2 if per >= 40 else 1
        if len(segs) > 2 * groups:          # chains of short streams: left whole
            R = 1
    if R > 1:
        cum = np.concatenate([[0], np.cumsum(SHARES_64THS[R])])
        assert cum[-1] == 64
        pieces, acc_of = [], {}
        n_g = {}
        for (p, b, c, k0, k1) in segs:
            n_g[p] = n_g.get(p, 0) + -(-(k1 - k0) // tile_n)
        for idx, (p, b, c, k0, k1) in enumerate(segs):
            nt = -(-(k1 - k0) // tile_n)
            acc = acc_of.get(p, 0)
            for r in range(R):
                lo = max(n_g[p] * int(cum[r]) // 64 - acc, 0)
                hi = min(n_g[p] * int(cum[r + 1]) // 64 - acc, nt)
                if lo < hi:
                    pieces.append((r * groups + p, b, c, k0 + lo * tile_n, min(k0 + hi * tile_n, k1), idx * R + r))
            acc_of[p] = acc + nt
        return groups, m_tiles, [q[:5] for q in pieces], [q[5] for q in pieces], R, len(segs)
    return groups, m_tiles, segs, list(range(len(segs))), 1, len(segs)


SHARES_64THS = {2: [52, 12], 4: [44, 10, 7, 3]}


def test_sub_bound_follows_the_published_shares():
    for R, shares in SHARES_64THS.items():
        cum = np.concatenate([[0], np.cumsum(shares)])
        for n in (0, 1, 7, 63, 64, 443, 16384, 10 ** 9):
            got = [bd.yoco_xattn_sub_bound(n, R, r) for r in range(R + 1)]
            assert got == [n * int(c) // 64 for c in cum] and got[0] == 0 and got[-1] == n
            assert all(x <= y for x, y in zip(got, got[1:]))
    assert [bd.yoco_xattn_sub_bound(100, 1, r) for r in (0, 1)] == [0, 100]
    assert bd.yoco_xattn_sub_bound(100, 3, 1) == -1 and bd.yoco_xattn_sub_bound(100, 8, 1) == -1
    assert bd.yoco_xattn_sub_bound(-1, 2, 1) == -1


CASES = [
    dict(B=128, Hq=8, Hkv=8, d=128, T=1, lens=[2048 + 16 * i for i in range(128)]),   # long groups of short streams
    dict(B=1, Hq=4, Hkv=1, d=64, T=1, lens=[512]),
    dict(B=1, Hq=32, Hkv=8, d=128, T=1, lens=[32768]),
    dict(B=1, Hq=32, Hkv=8, d=128, T=1, lens=[1048576]),
    dict(B=16, Hq=32, Hkv=8, d=128, T=1, lens=list(range(4096, 4096 + 16 * 7919, 7919))),
    dict(B=3, Hq=24, Hkv=8, d=128, T=2, lens=[1, 0, 65]),
    dict(B=2, Hq=32, Hkv=8, d=128, T=512, lens=[262656, 262656]),
    dict(B=2, Hq=32, Hkv=8, d=128, T=160, lens=[1160, 937]),
]


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("sm_count", [148, 7])
def test_plan_partitions_every_stream_exactly(case, sm_count):
    G = case["Hq"] // case["Hkv"]
    modes = [bd.MODE_CHUNK] + ([bd.MODE_DECODE] if G * case["T"] <= 16 else [])
    for mode in modes:
        shape = bd.make_shape(case["B"], case["Hq"], case["Hkv"], case["d"], case["T"])
        info, segs = bd.yoco_xattn_plan(shape, case["lens"], sm_count, mode)
        groups, m_tiles, want, want_slots, R, coarse = restated_plan(case["B"], case["Hkv"], case["lens"], sm_count,
                                                                     mode, G, case["T"])
        assert info.num_groups == groups and info.m_tiles == m_tiles
        assert info.num_ctas == groups * m_tiles
        assert info.sub_items == R and info.num_slots == coarse * R
        got = [(s.group, s.b, s.c, s.k_begin, s.k_end) for s in segs]
        assert got == want                                     # integer for integer
        assert [s.slot for s in segs] == want_slots            # unique, ascending, inside the workspace
        assert all(x < y for x, y in zip(want_slots, want_slots[1:])) and (not segs or segs[-1].slot < info.num_slots)
        # partition: no gap, no overlap, in order
        for b in range(case["B"]):
            for c in range(case["Hkv"]):
                mine = [s for s in segs if s.b == b and s.c == c]
                pos = 0
                for s in mine:
                    assert s.k_begin == pos and s.k_end > s.k_begin and s.k_begin % info.tile_n == 0
                    pos = s.k_end
                assert pos == case["lens"][b]
                if mine and R == 1:
                    assert [s.slot for s in mine] == list(range(mine[0].slot, mine[0].slot + len(mine)))
        # balance: every group streams the same number of tiles (+-1), all its pieces taken together
        tiles = {}
        for s in segs:
            tiles[s.group % groups] = tiles.get(s.group % groups, 0) + -(-(s.k_end - s.k_begin) // info.tile_n)
        if tiles:
            assert max(tiles.values()) - min(tiles.values()) <= 1
        # slots of one stream: a run of R per coarse segment
        per_stream = {}
        for s in segs:
            per_stream.setdefault((s.b, s.c), set()).add(s.slot // R)
        assert info.max_splits == R * max([0] + [len(v) for v in per_stream.values()])
        for v in per_stream.values():
            assert sorted(v) == list(range(min(v), min(v) + len(v)))
        # determinism
        info2, segs2 = bd.yoco_xattn_plan(shape, case["lens"], sm_count, mode)
        assert bytes(info) == bytes(info2) and [bytes(s) for s in segs] == [bytes(s) for s in segs2]
        assert bd.yoco_xattn_workspace_size(shape, case["lens"], mode, sm_count=sm_count) == info.workspace_bytes


def test_one_million_tokens_fills_the_machine_in_one_wave():
    shape = bd.make_shape(1, 32, 8, 128, 1)
    info, segs = bd.yoco_xattn_plan(shape, [1048576], 148, bd.MODE_DECODE)
    assert info.num_groups == 296 and info.total_tiles == 8 * 16384
    assert info.needs_combine == 1 and info.sub_items == 4 and info.num_segments == 4 * 296
    assert info.num_slots == 4 * 296
    # piece 0 of every group is the large one; the last pieces are 3/64 of the group
    sizes = {}
    for s in segs:
        sizes.setdefault(s.group // 296, []).append(s.k_end - s.k_begin)
    per_group = 1048576 * 8 / 296
    assert min(sizes[0]) >= 0.68 * per_group and max(sizes[3]) <= 0.05 * per_group


def test_unsplit_streams_need_no_combine():
    shape = bd.make_shape(400, 8, 8, 128, 1)
    info, _ = bd.yoco_xattn_plan(shape, [64] * 400, 148, bd.MODE_DECODE)
    assert info.needs_combine == 0 and info.max_splits == 1


@pytest.mark.parametrize("kw,code", [
    (dict(d=96), bd.ERR_UNSUPPORTED),
    (dict(Hq=30), bd.ERR_UNSUPPORTED),
    (dict(T=5), bd.ERR_UNSUPPORTED),           # G*T = 20 rows > 16 in decode mode
    (dict(T=0), bd.ERR_INVALID_ARG),
    (dict(B=-1), bd.ERR_INVALID_ARG),
    (dict(kv_head_stride=100), bd.ERR_UNSUPPORTED),
])
def test_bad_shapes_are_rejected_on_the_host(kw, code):
    args = dict(B=1, Hq=32, Hkv=8, d=128, T=1)
    args.update(kw)
    shape = bd.make_shape(**args)
    with pytest.raises(bd.YocoError) as e:
        bd.yoco_xattn_plan(shape, [100], 148, bd.MODE_DECODE)
    assert e.value.code == code


def test_negative_length_and_short_head_stride_are_invalid():
    shape = bd.make_shape(1, 8, 8, 128, 1)
    with pytest.raises(bd.YocoError) as e:
        bd.yoco_xattn_plan(shape, [-3], 148, bd.MODE_DECODE)
    assert e.value.code == bd.ERR_INVALID_ARG
    shape = bd.make_shape(1, 8, 8, 128, 1, kv_head_stride=128 * 10)
    with pytest.raises(bd.YocoError) as e:
        bd.yoco_xattn_plan(shape, [11], 148, bd.MODE_DECODE)
    assert e.value.code == bd.ERR_INVALID_ARG


def test_null_and_misaligned_pointers_fail_before_any_cuda_call():
    L = bd.lib()
    shape = bd.make_shape(1, 8, 8, 128, 1, max_kv_len=64)
    f = L.yoco_xattn_decode
    assert f(ctypes.byref(shape), None, None, None, None, None, None, None, None, 0, None) == bd.ERR_INVALID_ARG
    assert f(None, None, None, None, None, None, None, None, None, 0, None) == bd.ERR_INVALID_ARG
    p = ctypes.c_void_p
    assert f(ctypes.byref(shape), p(4096), p(4096 + 2), p(8192), None, None, p(4096), None, p(4096), 1 << 20,
             None) == bd.ERR_INVALID_ARG
    assert L.yoco_xattn_combine(4, 0, 128, None, None, None, None, None) == bd.ERR_INVALID_ARG
    assert L.yoco_xattn_combine(4, 2, 100, p(4096), p(4096), p(4096), None, None) == bd.ERR_UNSUPPORTED
    assert L.yoco_xattn_combine(4, 2, 128, None, p(4096), p(4096), None, None) == bd.ERR_INVALID_ARG


@pytest.mark.parametrize("case", [
    dict(B=1, Hq=32, Hkv=8, d=128, T=1, lens=[32768], C=1024),
    dict(B=3, Hq=8, Hkv=2, d=128, T=1, lens=[100, 5000, 63], C=130),
    dict(B=2, Hq=8, Hkv=2, d=128, T=40, lens=[4000, 41], C=300),
    dict(B=1, Hq=8, Hkv=2, d=128, T=4, lens=[1000], C=1),
    dict(B=1, Hq=8, Hkv=2, d=128, T=1, lens=[1000], C=5000),
])
def test_sliding_window_plan_skips_only_tiles_no_row_can_see(case):
    """With a window C the lowest key any row sees is that of row 0, (N - T) - C + 1; the plan
    starts at the tile that holds it and still partitions the rest exactly."""
    G, T, C = case["Hq"] // case["Hkv"], case["T"], case["C"]
    modes = [bd.MODE_CHUNK] + ([bd.MODE_DECODE] if G * T <= 16 else [])
    for mode in modes:
        shape = bd.make_shape(case["B"], case["Hq"], case["Hkv"], case["d"], T, window=C)
        info, segs = bd.yoco_xattn_plan(shape, case["lens"], 148, mode)
        want_total = 0
        for b, n in enumerate(case["lens"]):
            first_key = max(0, (n - T) - C + 1)
            start = min(first_key // info.tile_n, -(-n // info.tile_n)) * info.tile_n
            want_total += case["Hkv"] * (-(-n // info.tile_n) - start // info.tile_n)
            for c in range(case["Hkv"]):
                mine = [s for s in segs if s.b == b and s.c == c]
                pos = start
                for s in mine:
                    assert s.k_begin == pos and s.k_end > s.k_begin
                    pos = s.k_end
                assert pos == (n if mine else start) and (mine or start >= n or n == 0)
                assert start <= first_key < start + info.tile_n or n - T - C + 1 <= 0
        assert info.total_tiles == want_total
        tiles = {}
        for s in segs:
            tiles[s.group] = tiles.get(s.group, 0) + -(-(s.k_end - s.k_begin) // info.tile_n)
        if tiles:
            assert max(tiles.values()) - min(tiles.values()) <= 1


def test_negative_window_is_rejected():
    shape = bd.make_shape(1, 8, 8, 128, 1, window=-1)
    with pytest.raises(bd.YocoError) as e:
        bd.yoco_xattn_plan(shape, [100], 148, bd.MODE_DECODE)
    assert e.value.code == bd.ERR_INVALID_ARG


def test_new_entry_points_validate_arguments_before_touching_cuda():
    """Shape and pointer errors of the later entry points come back as codes on a box without a GPU."""
    L = bd.lib()
    p = ctypes.c_void_p
    ok_shape = bd.KvAppendShape(1, 8, 128, 1, 4096, 1e-6, 0)
    lens = np.array([4], dtype=np.int32)
    pl = p(lens.ctypes.data)
    assert L.yoco_kv_append(None, p(16), p(16), p(16), p(16), p(16), None, pl, None) == bd.ERR_INVALID_ARG
    for bad in (bd.KvAppendShape(1, 8, 128, 1, 4000, 1e-6, 0),        # d_model not a multiple of 128
                bd.KvAppendShape(1, 8, 96, 1, 4096, 1e-6, 0),         # head size
                bd.KvAppendShape(600, 8, 128, 1, 4096, 1e-6, 0)):     # too many sequences for the parameter table
        assert L.yoco_kv_append(ctypes.byref(bad), p(16), p(16), p(16), p(16), p(16), None, pl, None) == bd.ERR_UNSUPPORTED
    neg = bd.KvAppendShape(1, 8, 128, 1, 4096, -1.0, 0)
    assert L.yoco_kv_append(ctypes.byref(neg), p(16), p(16), p(16), p(16), p(16), None, pl, None) == bd.ERR_INVALID_ARG
    assert L.yoco_kv_append(ctypes.byref(ok_shape), None, p(16), p(16), p(16), p(16), None, pl, None) == bd.ERR_INVALID_ARG
    assert L.yoco_kv_fold_gain(-1, 8, p(16), p(16), p(32), None) == bd.ERR_INVALID_ARG
    assert L.yoco_kv_fold_gain(8, 8, p(16), p(32), p(32), None) == bd.ERR_INVALID_ARG      # Wg aliases W
    shape = bd.make_shape(1, 8, 8, 64, 1, max_kv_len=64)
    ones = np.ones(8, dtype=np.float32)
    po = p(ones.ctypes.data)
    assert L.yoco_xattn_decode_fp8(ctypes.byref(shape), p(16), p(16), p(16), po, po, None, None, p(16), None, p(256), 1 << 20,
                                   None) == bd.ERR_UNSUPPORTED                             # d = 64
    shape2 = bd.make_shape(1, 8, 8, 128, 2, max_kv_len=64)
    assert L.yoco_xattn_decode_partial(ctypes.byref(shape2), p(16), p(16), p(16), None, None, p(16), p(16), p(256),
                                       1 << 20, None) == bd.ERR_UNSUPPORTED                # T = 2
    assert L.yoco_xattn_combine_gathered(4, 0, 128, None, None, None, None, None) == bd.ERR_INVALID_ARG


def test_overlapping_offsets_and_a_stride_too_short_are_rejected_on_the_host():
    """Sequence i occupies Hkv * head_rows rows from token offset cu[i]; offsets that let the next
    sequence start inside it would make attention read a neighbour's keys and the cache write land in
    a neighbour's heads.  Both entry points must say so before any CUDA call."""
    L = bd.lib()
    p = ctypes.c_void_p
    lens = np.array([100, 50], dtype=np.int32)
    pl = p(lens.ctypes.data)

    def decode(shape, cu):
        cu = np.asarray(cu, dtype=np.int32)
        return L.yoco_xattn_decode(ctypes.byref(shape), p(4096), p(4096), p(4096), p(cu.ctypes.data), pl, p(4096),
                                   None, p(4096), 1 << 20, None)

    tight = bd.make_shape(2, 8, 8, 128, 1, max_kv_len=100)
    assert decode(tight, [0, 99, 150]) == bd.ERR_INVALID_ARG          # second sequence starts inside the first
    assert decode(tight, [0, 100, 149]) == bd.ERR_INVALID_ARG         # the last one does not fit its own range
    assert decode(tight, [0, 120, 100]) == bd.ERR_INVALID_ARG         # not monotone
    strided = bd.make_shape(2, 8, 8, 128, 1, kv_head_stride=128 * 128, max_kv_len=100)
    assert decode(strided, [0, 100, 228]) == bd.ERR_INVALID_ARG       # capacity 128 per head, offsets say 100
    short = bd.make_shape(2, 8, 8, 128, 1, kv_head_stride=64 * 128, max_kv_len=100)
    assert decode(short, [0, 128, 256]) == bd.ERR_INVALID_ARG         # stride shorter than the first sequence
    # the same offsets are fine once they leave room (no GPU here: the call then fails later, at the device query)
    assert decode(tight, [0, 100, 150]) != bd.ERR_INVALID_ARG
    assert decode(strided, [0, 128, 256]) != bd.ERR_INVALID_ARG

    ash = bd.KvAppendShape(2, 8, 128, 1, 4096, 1e-6, 0)

    def append(shape, cu):
        cu = np.asarray(cu, dtype=np.int32)
        return L.yoco_kv_append(ctypes.byref(shape), p(16), p(16), p(16), p(16), p(16), p(cu.ctypes.data), pl, None)

    assert append(ash, [0, 99, 150]) == bd.ERR_INVALID_ARG
    assert append(ash, [0, 100, 149]) == bd.ERR_INVALID_ARG
    assert append(bd.KvAppendShape(2, 8, 128, 1, 4096, 1e-6, 128 * 128), [0, 100, 228]) == bd.ERR_INVALID_ARG
    assert append(ash, [0, 100, 150]) != bd.ERR_INVALID_ARG


@pytest.mark.parametrize("T,C", [(1, 0), (5, 0), (1, 300), (7, 300), (40, 1), (3, 100000)])
def test_plan_of_a_key_shard_covers_exactly_the_keys_some_row_sees(T, C):
    """A shard holds keys [off, off + n) of a sequence of N keys; query row t sits at position N - T + t
    of the whole sequence.  The plan of the shard must cover, tile by tile, exactly the local keys from
    the tile of the lowest key row 0 sees up to the last key the last row sees, for every KV head --
    restated here from the mask inequalities, not from the planner's code."""
    N = 20000
    mode = bd.MODE_DECODE if T * 2 <= 16 else bd.MODE_CHUNK
    tile = 64 if mode == bd.MODE_DECODE else 128
    shape = bd.make_shape(3, 4, 2, 128, T, window=C)
    shards = [(0, 7000), (7000, 9000), (16000, 4000)]          # (offset, count) of the three "sequences"
    lens = [n for _, n in shards]
    offs = [o for o, _ in shards]
    info, segs = bd.yoco_xattn_plan_at(shape, lens, offs, [N] * 3, 148, mode)
    for b, (off, n) in enumerate(shards):
        pos0, pos_last = N - T, N - 1                          # whole-sequence positions of the first / last row
        lo_seen = max(pos0 - C + 1, 0) if C > 0 else 0         # lowest whole-sequence key row 0 sees
        first = max(lo_seen - off, 0)                          # ... as a local key
        last = min(pos_last - off, n - 1)                      # highest local key the last row sees
        for c in range(2):
            mine = sorted((s.k_begin, s.k_end) for s in segs if s.b == b and s.c == c)
            if last < first:
                assert mine == []
                continue
            assert mine[0][0] == first // tile * tile and mine[-1][1] == last + 1
            for (a0, a1), (b0, b1) in zip(mine, mine[1:]):
                assert a1 == b0 and a1 % tile == 0
    # offsets and totals come together, and a shard may not reach past its sequence
    L = bd.lib()
    p = ctypes.c_void_p
    a = np.array(lens, dtype=np.int32)
    o = np.array(offs, dtype=np.int32)
    t_bad = np.array([N, N, 19999], dtype=np.int32)
    pi = bd.PlanInfo()
    assert L.yoco_xattn_plan_at(ctypes.byref(shape), p(a.ctypes.data), p(o.ctypes.data), None, 148, mode,
                                ctypes.byref(pi), None, 0) == bd.ERR_INVALID_ARG
    assert L.yoco_xattn_plan_at(ctypes.byref(shape), p(a.ctypes.data), p(o.ctypes.data), p(t_bad.ctypes.data), 148, mode,
                                ctypes.byref(pi), None, 0) == bd.ERR_INVALID_ARG


def test_status_word_names_the_wait_and_the_cta():
    """0 is ok; otherwise the low byte is the kind of wait that ran out and the rest 1 + the CTA."""
    assert bd.yoco_xattn_decode_status_word(0) == (bd.OK, 0, -1)
    for wc in (bd.WAIT_ITEM_QUEUE, bd.WAIT_RING_FULL, bd.WAIT_RING_EMPTY, bd.WAIT_TENSOR, bd.WAIT_DRAIN,
               bd.WAIT_MISALIGNED):
        for cta in (0, 1, 147, 295, 70000):
            word = wc | ((cta + 1) << 8)
            assert bd.yoco_xattn_decode_status_word(word) == (bd.ERR_TIMEOUT, wc, cta)
    # either output may be omitted
    assert bd.lib().yoco_xattn_decode_status_word(2 | (5 << 8), None, None) == bd.ERR_TIMEOUT
    # the header's names carry the same numbers
    hdr = open(os.path.join(ROOT, "include", "yoco_xattn.h")).read()
    for name, val in (("ITEM_QUEUE", 1), ("RING_FULL", 2), ("RING_EMPTY", 3), ("TENSOR", 4), ("DRAIN", 5),
                      ("MISALIGNED", 6)):
        assert re.search(rf"#define YOCO_WAIT_{name}\s+{val}\b", hdr), name
    p = ctypes.c_void_p
    shape = bd.make_shape(1, 8, 8, 128, 1, max_kv_len=64)
    f = bd.lib().yoco_xattn_selftest_wait_expiry
    for bad_limit in (0, -5, 1001):
        assert f(ctypes.byref(shape), p(4096), p(4096), p(4096), None, None, p(4096), p(4096), 1 << 20, bad_limit,
                 None) == bd.ERR_INVALID_ARG


def test_public_header_is_plain_c_and_cxx(tmp_path):
    """The boundary is a C ABI: the header must compile on its own as C99 and as C++11, warnings
    as errors, and a C program must be able to link the planner (a pure host call) from the library."""
    import shutil
    import subprocess
    inc = os.path.join(ROOT, "include")
    src = tmp_path / "use.c"
    src.write_text('#include "yoco_xattn.h"\n#include <stdio.h>\n#include <string.h>\n'
                   'int main(void) {\n'
                   '    yoco_xattn_shape s;\n    yoco_xattn_plan_info info;\n    int32_t len = 1048576;\n'
                   '    memset(&s, 0, sizeof s);\n'
                   '    s.B = 1; s.Hq = 32; s.Hkv = 8; s.d = 128; s.T = 1; s.max_kv_len = len;\n'
                   '    int32_t rc = yoco_xattn_plan(&s, &len, 148, YOCO_MODE_DECODE, &info, 0, 0);\n'
                   '    printf("%d %d %d %d\\n", (int)rc, (int)info.num_groups, (int)info.sub_items, (int)info.num_slots);\n'
                   '    return rc;\n}\n')
    for cc, std in (("gcc", "-std=c99"), ("g++", "-std=c++11")):
        if shutil.which(cc) is None:
            pytest.skip(f"{cc} not installed")
        lang = ["-x", "c++"] if cc == "g++" else []
        subprocess.run([cc, std, "-Wall", "-Wextra", "-Werror", "-pedantic", "-fsyntax-only", "-I", inc] + lang + [str(src)],
                       check=True)
    exe = tmp_path / "use"
    libdir, libname = os.path.split(bd.LIB_PATH)
    subprocess.run(["gcc", "-std=c99", "-I", inc, str(src), "-o", str(exe), os.path.join(libdir, libname),
                    f"-Wl,-rpath,{libdir}"], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()
    assert out == ["0", "296", "4", "1184"]
