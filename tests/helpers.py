"""Shared test plumbing: run the CUDA path through the C ABI and compare with the oracle."""
import numpy as np

import synth_inputs as si

MAX_ABS_TOL = 1e-2     # bf16 in, fp32 accumulate: max-abs 1e-2 and relative L2 5e-3 against the fp64 oracle
REL_L2_TOL = 5e-3
LSE_ABS_TOL = 2e-3
GUARD = 4096           # sentinel elements on both sides of every output buffer


def to_dev_bf16(bits: np.ndarray):
    import torch
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def bf16_dev_to_f64(t) -> np.ndarray:
    import torch
    bits = t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    return si.bf16_bits_to_f32(bits).astype(np.float64)


def errors(got: np.ndarray, ref: np.ndarray):
    diff = got.astype(np.float64) - ref
    max_abs = float(np.abs(diff).max()) if diff.size else 0.0
    denom = float(np.linalg.norm(ref.ravel()))
    rel_l2 = float(np.linalg.norm(diff.ravel()) / denom) if denom > 0 else float(np.linalg.norm(diff.ravel()))
    return max_abs, rel_l2


def assert_close(got, ref, what=""):
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    max_abs, rel_l2 = errors(got, ref)
    assert max_abs <= MAX_ABS_TOL, f"{what}: max-abs {max_abs:.3e} > {MAX_ABS_TOL}"
    assert rel_l2 <= REL_L2_TOL, f"{what}: rel-L2 {rel_l2:.3e} > {REL_L2_TOL}"
    return max_abs, rel_l2


def assert_lse_close(got, ref, what=""):
    inf_ref = np.isneginf(ref)
    assert (np.isneginf(got) == inf_ref).all(), f"{what}: -inf pattern of LSE differs"
    if (~inf_ref).any():
        err = np.abs(got[~inf_ref].astype(np.float64) - ref[~inf_ref]).max()
        assert err <= LSE_ABS_TOL, f"{what}: LSE error {err:.3e}"


class GpuRunner:
    """Holds device copies of K/V and runs decode / chunk calls through the binding."""

    def __init__(self, B, Hq, Hkv, d, T, kv_len, K_bits, V_bits, cu=None, kv_head_stride=0, scale=0.0, window=0):
        import torch
        from paper_2405_05254_b200 import binding
        self.torch, self.bd = torch, binding
        self.B, self.Hq, self.Hkv, self.d, self.T = B, Hq, Hkv, d, T
        self.kv_len = np.asarray(kv_len, dtype=np.int32)
        self.cu = None if cu is None else np.asarray(cu, dtype=np.int32)
        self.shape = binding.make_shape(B, Hq, Hkv, d, T, scale=scale, kv_head_stride=kv_head_stride,
                                        max_kv_len=int(self.kv_len.max()) if B else 0, window=window)
        self.K = to_dev_bf16(K_bits.reshape(-1))
        self.V = to_dev_bf16(V_bits.reshape(-1))

    def _buffers(self, mode):
        torch = self.torch
        n = self.B * self.Hq * self.T
        self.o_buf = torch.full((GUARD + n * self.d + GUARD,), 777.0, dtype=torch.bfloat16, device="cuda")
        self.l_buf = torch.full((GUARD + n + GUARD,), 777.0, dtype=torch.float32, device="cuda")
        ws_bytes = self.bd.yoco_xattn_workspace_size(self.shape, self.kv_len, mode)
        self.ws = torch.full((ws_bytes + 2 * GUARD,), 0x5A, dtype=torch.uint8, device="cuda")
        O = self.o_buf[GUARD:GUARD + n * self.d]
        L = self.l_buf[GUARD:GUARD + n]
        W = self.ws[GUARD:GUARD + ws_bytes]
        assert W.data_ptr() % 256 == 0
        return O, L, W

    def _check_guards(self):
        torch = self.torch
        for buf in (self.o_buf, self.l_buf):
            assert (buf[:GUARD] == 777.0).all() and (buf[-GUARD:] == 777.0).all(), "guard band overwritten"
        assert (self.ws[:GUARD] == 0x5A).all() and (self.ws[-GUARD:] == 0x5A).all(), "workspace guard overwritten"

    def run(self, Q_bits, mode="decode", want_lse=True):
        bd = self.bd
        m = bd.MODE_DECODE if mode == "decode" else bd.MODE_CHUNK
        O, L, W = self._buffers(m)
        Q = to_dev_bf16(Q_bits.reshape(-1))
        fn = bd.yoco_xattn_decode if mode == "decode" else bd.yoco_xattn_chunk
        fn(self.shape, Q, self.K, self.V, self.cu, self.kv_len, O, L if want_lse else None, W)
        rc = bd.yoco_xattn_status(W)
        assert rc == 0, f"device status {rc}"
        self._check_guards()
        o = bf16_dev_to_f64(O).reshape(self.B, self.Hq, self.T, self.d)
        lse = L.cpu().numpy().reshape(self.B, self.Hq, self.T)
        return o, lse, O
