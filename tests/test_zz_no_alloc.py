"""The workspace-free decode entry point (collected last on purpose).

Some users of this library cannot create device memory where they call attention: a plugin
running inside an application that owns the allocator, or a serving loop that has frozen its
memory pool.  ``yoco_xattn_decode_static`` serves them from a 4 MiB buffer compiled into the
library.  It must give the oracle's result (and the same as ``yoco_xattn_decode`` with a caller
workspace), on the first call and on later calls that find the buffer full of the previous call's
tables and partials; it must leave the amount of free device memory exactly as it found it; and its
status word must be readable although the caller never sees the buffer.
"""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from helpers import MAX_ABS_TOL, REL_L2_TOL, assert_close, assert_lse_close, errors, to_dev_bf16, bf16_dev_to_f64

pytestmark = pytest.mark.gpu


class Problem:
    """Inputs, outputs and the oracle's answer of one decode problem, created before any measured call."""

    def __init__(self, w, layer):
        import torch
        from paper_2405_05254_b200 import binding as bd
        self.w = w
        Kb, Vb, Qb = w.make_k(), w.make_v(), w.make_q(layer)
        self.K, self.V, self.Q = to_dev_bf16(Kb), to_dev_bf16(Vb), to_dev_bf16(Qb.reshape(-1))
        self.shape = bd.make_shape(w.B, w.Hq, w.Hkv, w.d, w.T, max_kv_len=int(w.kv_len.max()))
        n = w.B * w.Hq * w.T
        self.ws = torch.empty(bd.yoco_xattn_workspace_size(self.shape, w.kv_len, bd.MODE_DECODE), dtype=torch.uint8,
                              device="cuda")
        self.O_ws = torch.empty(n * w.d, dtype=torch.bfloat16, device="cuda")
        self.L_ws = torch.empty(n, dtype=torch.float32, device="cuda")
        self.O = torch.full((n * w.d,), 123.0, dtype=torch.bfloat16, device="cuda")
        self.L = torch.full((n,), 123.0, dtype=torch.float32, device="cuda")
        self.o_ref, self.lse_ref = oracle.xattn(Qb, Kb, Vb, w.cu, w.kv_len, B=w.B, Hq=w.Hq, Hkv=w.Hkv, d=w.d, T=w.T)

    def run_static(self):
        from paper_2405_05254_b200 import binding as bd
        bd.yoco_xattn_decode_static(self.shape, self.Q, self.K, self.V, self.w.cu, self.w.kv_len, self.O, self.L)

    def check(self):
        import torch
        from paper_2405_05254_b200 import binding as bd
        w = self.w
        assert bd.yoco_xattn_status(None) == 0          # the status word inside the built-in buffer
        torch.cuda.synchronize()
        got = bf16_dev_to_f64(self.O).reshape(self.o_ref.shape)
        assert_close(got, self.o_ref, f"static scratch, {w.name}")
        assert_lse_close(self.L.cpu().numpy().reshape(self.lse_ref.shape), self.lse_ref, f"static scratch, {w.name}")
        # and it is the same computation as the entry point with a caller workspace
        bd.yoco_xattn_decode(self.shape, self.Q, self.K, self.V, w.cu, w.kv_len, self.O_ws, self.L_ws, self.ws)
        assert bd.yoco_xattn_status(self.ws) == 0
        max_abs, rel_l2 = errors(got, bf16_dev_to_f64(self.O_ws).reshape(self.o_ref.shape))
        assert max_abs <= MAX_ABS_TOL and rel_l2 <= REL_L2_TOL, (w.name, max_abs, rel_l2)
        assert np.abs(self.L.cpu().numpy() - self.L_ws.cpu().numpy()).max() <= 2e-3


def test_static_scratch_decode_matches_the_oracle_on_calls_in_a_row_and_allocates_nothing():
    import torch
    # first call: one long sequence cut into many splits; second call: a ragged batch whose tables and
    # partial slots land on top of the first call's leftovers; third: the first shape again
    long_seq = dict(B=1, Hq=32, Hkv=8, d=128, T=1, seed=21, kv_len=[40000])
    problems = [Problem(si.Workload("static_a", layers=1, **long_seq), 0),
                Problem(si.workload("ragged_small"), 0),
                Problem(si.Workload("static_a", layers=2, **long_seq), 1)]
    problems[0].run_static()                             # first call on the device: looks the buffer up
    problems[0].check()
    for p in problems[1:]:
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        p.run_static()
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before, "the workspace-free entry point changed free memory"
        p.check()


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
