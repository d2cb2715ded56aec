"""Key-range sharding through the C ABI on one GPU: the ranks' calls run one after another (no
kernel waits for another), each on its own cut of the cache; the gathered partials are merged with
yoco_xattn_combine_gathered and must equal the oracle's unsharded attention."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from helpers import LSE_ABS_TOL, assert_close, assert_lse_close, bf16_dev_to_f64, to_dev_bf16

pytestmark = pytest.mark.gpu


def sharded_decode(w, world, layer=0):
    import torch
    from paper_2405_05254_b200 import binding as bd, shard
    K, V, Qb = w.make_k(), w.make_v(), w.make_q(layer)
    Q = to_dev_bf16(Qb.reshape(-1))
    rows = w.B * w.Hq
    off, cnt = shard.key_range_shards(w.kv_len, world)
    all_o = torch.full((world, rows, w.d), 7.0, dtype=torch.float32, device="cuda")
    all_l = torch.full((world, rows), 7.0, dtype=torch.float32, device="cuda")
    parts = []
    for r in range(world):
        Kr = shard.take_key_range(K, w.kv_len, w.Hkv, w.d, off[r], cnt[r])
        Vr = shard.take_key_range(V, w.kv_len, w.Hkv, w.d, off[r], cnt[r])
        # an all-empty shard still needs valid (16-byte aligned) K/V pointers
        Kd = to_dev_bf16(Kr if Kr.size else np.zeros(8, dtype=np.uint16))
        Vd = to_dev_bf16(Vr if Vr.size else np.zeros(8, dtype=np.uint16))
        shape = bd.make_shape(w.B, w.Hq, w.Hkv, w.d, 1, max_kv_len=int(cnt[r].max()))
        ws = torch.empty(bd.yoco_xattn_workspace_size(shape, cnt[r], bd.MODE_DECODE), dtype=torch.uint8, device="cuda")
        bd.yoco_xattn_decode_partial(shape, Q, Kd, Vd, None, cnt[r], all_o[r], all_l[r], ws)
        assert bd.yoco_xattn_status(ws) == 0
        parts.append((Kr, Vr, cnt[r]))
    O = torch.empty(rows * w.d, dtype=torch.bfloat16, device="cuda")
    L = torch.empty(rows, dtype=torch.float32, device="cuda")
    bd.yoco_xattn_combine_gathered(all_o, all_l, O, L)
    torch.cuda.synchronize()
    return (bf16_dev_to_f64(O).reshape(w.B, w.Hq, 1, w.d), L.cpu().numpy().reshape(w.B, w.Hq, 1),
            all_o.cpu().numpy(), all_l.cpu().numpy(), parts, (Qb, K, V))


@pytest.mark.parametrize("world", [1, 2, 3, 8])
def test_sharded_decode_merges_to_the_unsharded_attention(world):
    w = si.Workload("shard", B=4, Hq=32, Hkv=8, d=128, T=1, layers=1, seed=61, kv_len=[5000, 64, 700, 1])
    o, lse, all_o, all_l, parts, (Q, K, V) = sharded_decode(w, world)
    o_ref, lse_ref = oracle.xattn(Q, K, V, w.cu, w.kv_len, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=1)
    assert_close(o, o_ref, f"sharded x{world}")
    assert_lse_close(lse, lse_ref, f"sharded x{world}")
    # each rank's partial is the attention over its own keys: normalised rows, natural-log LSE,
    # zeros and -inf where the rank holds nothing of a sequence
    for r, (Kr, Vr, cnt) in enumerate(parts):
        cu = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int32)
        po, pl = oracle.xattn(Q, Kr, Vr, cu, cnt, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=1)
        got_l = all_l[r].reshape(w.B, w.Hq, 1)
        assert (np.isneginf(got_l) == np.isneginf(pl)).all()
        live = ~np.isneginf(pl)
        assert np.abs(got_l[live] - pl[live]).max() <= LSE_ABS_TOL
        assert np.abs(all_o[r].reshape(w.B, w.Hq, 1, w.d) - po).max() <= 1e-2
        assert (all_o[r].reshape(w.B, w.Hq, w.d)[~live[..., 0]] == 0).all()


def sharded_at(w, world, mode, window=0, layer=0):
    """Every rank's call with the shard's place in the sequence (any T, any window), gathered and merged."""
    import torch
    from paper_2405_05254_b200 import binding as bd, shard
    K, V, Qb = w.make_k(), w.make_v(), w.make_q(layer)
    Q = to_dev_bf16(Qb.reshape(-1))
    rows = w.B * w.Hq * w.T
    tile = 64 if mode == "decode" else 128
    m = bd.MODE_DECODE if mode == "decode" else bd.MODE_CHUNK
    off, cnt = shard.key_range_shards(w.kv_len, world, tile=tile)
    all_o = torch.full((world, rows, w.d), 7.0, dtype=torch.float32, device="cuda")
    all_l = torch.full((world, rows), 7.0, dtype=torch.float32, device="cuda")
    for r in range(world):
        Kr = shard.take_key_range(K, w.kv_len, w.Hkv, w.d, off[r], cnt[r])
        Vr = shard.take_key_range(V, w.kv_len, w.Hkv, w.d, off[r], cnt[r])
        Kd = to_dev_bf16(Kr if Kr.size else np.zeros(8, dtype=np.uint16))
        Vd = to_dev_bf16(Vr if Vr.size else np.zeros(8, dtype=np.uint16))
        shape = bd.make_shape(w.B, w.Hq, w.Hkv, w.d, w.T, max_kv_len=int(cnt[r].max()), window=window)
        ws = torch.empty(bd.yoco_xattn_workspace_size_at(shape, cnt[r], off[r], w.kv_len, m), dtype=torch.uint8,
                         device="cuda")
        bd.yoco_xattn_partial_at(shape, Q, Kd, Vd, None, cnt[r], off[r], w.kv_len, all_o[r], all_l[r], ws, mode=m)
        assert bd.yoco_xattn_status(ws) == 0
    O = torch.empty(rows * w.d, dtype=torch.bfloat16, device="cuda")
    L = torch.empty(rows, dtype=torch.float32, device="cuda")
    bd.yoco_xattn_combine_gathered(all_o, all_l, O, L)
    torch.cuda.synchronize()
    o_ref, lse_ref = oracle.xattn(Qb, K, V, w.cu, w.kv_len, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=w.T, window=window)
    assert_close(bf16_dev_to_f64(O).reshape(o_ref.shape), o_ref, f"{mode} x{world} T={w.T} C={window}")
    assert_lse_close(L.cpu().numpy().reshape(lse_ref.shape), lse_ref, f"{mode} x{world} T={w.T} C={window}")
    return all_l.cpu().numpy()


@pytest.mark.parametrize("world,T,window", [(2, 2, 0), (3, 4, 0), (3, 1, 700), (4, 2, 129), (2, 3, 1)])
def test_sharded_decode_with_several_rows_and_windows(world, T, window):
    """Rows of a sharded call sit at their positions in the WHOLE sequence: the causal edge falls into
    the last shard only, a window may start in any shard, and shards wholly outside a row's window
    contribute -inf.  Merged result against the oracle on the unsharded cache."""
    w = si.Workload("shard_t", B=4, Hq=8, Hkv=2, d=128, T=T, layers=1, seed=62, kv_len=[5000, 64 + T, 700, T])
    all_l = sharded_at(w, world, "decode", window)
    if window and window < 600:
        assert np.isneginf(all_l[0].reshape(w.B, w.Hq, T)[0]).all()     # first shard of the long sequence: out of every window


@pytest.mark.parametrize("world,T,window", [(2, 40, 0), (3, 200, 0), (2, 130, 300), (3, 64, 2000)])
def test_sharded_chunk_through_the_tensor_core_path(world, T, window):
    w = si.Workload("shard_c", B=2, Hq=8, Hkv=2, d=128, T=T, layers=1, seed=63, kv_len=[3000 + T, 517 + T])
    sharded_at(w, world, "chunk", window)


def test_partial_entry_rejects_several_rows_and_windows():
    import torch
    from paper_2405_05254_b200 import binding as bd
    t = torch.zeros(64 * 128, dtype=torch.bfloat16, device="cuda")
    f = torch.zeros(4 * 128, dtype=torch.float32, device="cuda")
    for shape in (bd.make_shape(1, 1, 1, 128, 2, max_kv_len=64), bd.make_shape(1, 1, 1, 128, 1, max_kv_len=64, window=8)):
        with pytest.raises(bd.YocoError) as e:
            bd.yoco_xattn_decode_partial(shape, t, t, t, None, [64], f, f, t)
        assert e.value.code == bd.ERR_UNSUPPORTED
