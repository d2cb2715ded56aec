"""A bounded device-side wait that runs out, in the one safe form: nothing is in flight.

``yoco_xattn_selftest_wait_expiry`` runs the real decode kernel with a producer that starts no copy
and a wait limit of a few milliseconds.  The consumer warps' first wait for a tile then runs out, the
CTAs record which wait it was and leave in the ordinary way (no trap, no fault, no unbounded wait);
the host reads YOCO_ERR_TIMEOUT with the wait class and a CTA index, and the very next ordinary call
on the same GPU and the same workspace must pass parity against the oracle."""
import time

import numpy as np
import pytest

import oracle
import synth_inputs as si
from helpers import assert_close, assert_lse_close, bf16_dev_to_f64, to_dev_bf16

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("lens", [[3000, 1217], [70000]])
def test_expired_wait_is_reported_and_the_next_call_is_correct(lens):
    import torch
    from paper_2405_05254_b200 import binding as bd
    w = si.Workload("expiry", B=len(lens), Hq=32, Hkv=8, d=128, T=1, layers=1, seed=71, kv_len=lens)
    Kb, Vb, Qb = w.make_k(), w.make_v(), w.make_q(0)
    K, V, Q = to_dev_bf16(Kb), to_dev_bf16(Vb), to_dev_bf16(Qb.reshape(-1))
    shape = bd.make_shape(w.B, w.Hq, w.Hkv, w.d, w.T, max_kv_len=int(w.kv_len.max()))
    n = w.B * w.Hq
    ws = torch.empty(bd.yoco_xattn_workspace_size(shape, w.kv_len, bd.MODE_DECODE), dtype=torch.uint8, device="cuda")
    O = torch.zeros(n * w.d, dtype=torch.bfloat16, device="cuda")
    L = torch.zeros(n, dtype=torch.float32, device="cuda")
    sm = torch.cuda.get_device_properties(0).multi_processor_count
    info, _ = bd.yoco_xattn_plan(shape, w.kv_len, sm, bd.MODE_DECODE)

    t0 = time.perf_counter()
    bd.yoco_xattn_selftest_wait_expiry(shape, Q, K, V, w.cu, w.kv_len, O, ws, limit_ms=20)
    rc, wait_class, cta = bd.yoco_xattn_status_detail(ws)
    dt = time.perf_counter() - t0
    assert rc == bd.ERR_TIMEOUT
    assert wait_class == bd.WAIT_RING_FULL, wait_class          # a consumer waiting for a tile that nobody loads
    assert 0 <= cta < info.num_groups
    assert bd.yoco_xattn_status(ws) == bd.ERR_TIMEOUT            # the word stays until the next call clears it
    assert 0.015 < dt < 2.0, dt                                  # the limit was honoured, and only once per CTA
    assert torch.cuda.is_available() and int(torch.zeros(1, device="cuda").item()) == 0   # the context is alive

    # the same workspace, an ordinary call: status clean, result equal to the oracle's
    bd.yoco_xattn_decode(shape, Q, K, V, w.cu, w.kv_len, O, L, ws)
    assert bd.yoco_xattn_status_detail(ws) == (bd.OK, 0, -1)
    o_ref, lse_ref = oracle.xattn(Qb, Kb, Vb, w.cu, w.kv_len, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=w.T)
    assert_close(bf16_dev_to_f64(O).reshape(o_ref.shape), o_ref, "call after an expired wait")
    assert_lse_close(L.cpu().numpy().reshape(lse_ref.shape), lse_ref, "call after an expired wait")


def test_expired_wait_in_the_8_bit_decode_kernel_is_reported_and_the_next_call_is_correct():
    """The consumer warps of the 8-bit decode kernel take every fourth tile and first wait for the producer
    to have armed their tile; with a producer that arms nothing that wait runs out (the item-queue class),
    the CTAs leave in the ordinary way, and the next ordinary call on the same workspace matches the oracle."""
    import torch
    from paper_2405_05254_b200 import binding as bd
    w = si.Workload("expiry8", B=2, Hq=32, Hkv=8, d=128, T=1, layers=1, seed=72, kv_len=[9000, 2500])
    K8, V8, ks, vs = w.make_kv_fp8()
    Qb = w.make_q(0)
    K, V, Q = torch.from_numpy(K8).cuda(), torch.from_numpy(V8).cuda(), to_dev_bf16(Qb.reshape(-1))
    shape = bd.make_shape(w.B, w.Hq, w.Hkv, w.d, w.T, max_kv_len=int(w.kv_len.max()))
    n = w.B * w.Hq
    ws = torch.empty(bd.yoco_xattn_workspace_size(shape, w.kv_len, bd.MODE_DECODE), dtype=torch.uint8, device="cuda")
    O = torch.zeros(n * w.d, dtype=torch.bfloat16, device="cuda")
    L = torch.zeros(n, dtype=torch.float32, device="cuda")
    sm = torch.cuda.get_device_properties(0).multi_processor_count
    info, _ = bd.yoco_xattn_plan(shape, w.kv_len, sm, bd.MODE_DECODE)

    t0 = time.perf_counter()
    bd.yoco_xattn_selftest_wait_expiry_fp8(shape, Q, K, V, ks, vs, w.cu, w.kv_len, O, ws, limit_ms=20)
    rc, wait_class, cta = bd.yoco_xattn_status_detail(ws)
    dt = time.perf_counter() - t0
    assert rc == bd.ERR_TIMEOUT
    assert wait_class == bd.WAIT_ITEM_QUEUE, wait_class         # a consumer waiting for a tile that nobody arms
    assert 0 <= cta < info.num_groups
    assert 0.015 < dt < 2.0, dt
    assert int(torch.zeros(1, device="cuda").item()) == 0        # the context is alive

    bd.yoco_xattn_decode_fp8(shape, Q, K, V, ks, vs, w.cu, w.kv_len, O, L, ws)
    assert bd.yoco_xattn_status_detail(ws) == (bd.OK, 0, -1)
    o_ref, lse_ref = oracle.xattn_fp8(Qb, K8, V8, ks, vs, w.cu, w.kv_len, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=w.T)
    assert_close(bf16_dev_to_f64(O).reshape(o_ref.shape), o_ref, "8-bit call after an expired wait")
    assert_lse_close(L.cpu().numpy().reshape(lse_ref.shape), lse_ref, "8-bit call after an expired wait")
