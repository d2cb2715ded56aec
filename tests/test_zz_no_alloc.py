"""The workspace-free decode entry point (collected last on purpose).

Some users of this library cannot create device memory where they call attention: a plugin
running inside an application that owns the allocator, or a serving loop that has frozen its
memory pool.  ``yoco_xattn_decode_static`` serves them from a 4 MiB buffer compiled into the
library.  It must give the same result as ``yoco_xattn_decode`` with a caller workspace, on the
first call and on a second call that finds the buffer full of the first call's tables and partials.
"""
import numpy as np
import pytest

import synth_inputs as si
from helpers import MAX_ABS_TOL, REL_L2_TOL, errors, to_dev_bf16, bf16_dev_to_f64

pytestmark = pytest.mark.gpu


def _both_ways(w, layer):
    import torch
    from paper_2405_05254_b200 import binding as bd
    K, V, Q = to_dev_bf16(w.make_k()), to_dev_bf16(w.make_v()), to_dev_bf16(w.make_q(layer).reshape(-1))
    shape = bd.make_shape(w.B, w.Hq, w.Hkv, w.d, w.T, max_kv_len=int(w.kv_len.max()))
    n = w.B * w.Hq * w.T
    ws = torch.empty(bd.yoco_xattn_workspace_size(shape, w.kv_len, bd.MODE_DECODE), dtype=torch.uint8, device="cuda")
    O_ref = torch.empty(n * w.d, dtype=torch.bfloat16, device="cuda")
    L_ref = torch.empty(n, dtype=torch.float32, device="cuda")
    bd.yoco_xattn_decode(shape, Q, K, V, w.cu, w.kv_len, O_ref, L_ref, ws)
    assert bd.yoco_xattn_status(ws) == 0
    O = torch.full((n * w.d,), 123.0, dtype=torch.bfloat16, device="cuda")
    L = torch.full((n,), 123.0, dtype=torch.float32, device="cuda")
    bd.yoco_xattn_decode_static(shape, Q, K, V, w.cu, w.kv_len, O, L)
    torch.cuda.synchronize()
    got, ref = bf16_dev_to_f64(O), bf16_dev_to_f64(O_ref)
    max_abs, rel_l2 = errors(got, ref)
    assert max_abs <= MAX_ABS_TOL and rel_l2 <= REL_L2_TOL, (w.name, max_abs, rel_l2)
    assert np.abs(L.cpu().numpy() - L_ref.cpu().numpy()).max() <= 2e-3


def test_static_scratch_decode_matches_workspace_decode_on_two_calls_in_a_row():
    # first call: one long sequence cut into many splits; second call: a ragged batch whose
    # tables and partial slots land on top of the first call's leftovers
    _both_ways(si.Workload("static_a", B=1, Hq=32, Hkv=8, d=128, T=1, layers=1, seed=21, kv_len=[40000]), 0)
    _both_ways(si.workload("ragged_small"), 0)
    _both_ways(si.Workload("static_a", B=1, Hq=32, Hkv=8, d=128, T=1, layers=2, seed=21, kv_len=[40000]), 1)


def test_static_scratch_refuses_problems_beyond_its_size():
    import torch
    from paper_2405_05254_b200 import binding as bd
    B = 1200                                  # ~1500 segments x 16 rows x 129 floats > 4 MiB
    shape = bd.make_shape(B, 16, 1, 128, 1, max_kv_len=64)
    lens = np.full(B, 64, dtype=np.int32)
    assert bd.yoco_xattn_workspace_size(shape, lens, bd.MODE_DECODE) > bd.yoco_xattn_static_scratch_bytes()
    t = torch.zeros(B * 64 * 128, dtype=torch.bfloat16, device="cuda")
    q = torch.zeros(B * 16 * 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(bd.YocoError) as e:
        bd.yoco_xattn_decode_static(shape, q, t, t, None, lens, q.clone(), None)
    assert e.value.code == bd.ERR_STATIC_SCRATCH_EXCEEDED
    assert "static" in str(e.value)
