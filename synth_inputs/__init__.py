"""Seeded synthetic inputs for the cross-attention path (no attention arithmetic here).

The tests, ``bench.py`` and the smoke check draw every tensor from the counter-based
generator in ``gen.c`` so that the CUDA path and the CPU oracle are fed identical
bf16 bits.  Arrays are numpy ``uint16`` (bf16 bit patterns).

The five workloads mirror the long-context inference profiling set-up of the
paper (3B-class shapes, head dimension 128, 8 KV heads, contexts from 32K to 1M
tokens, Section 4.4 / Section 4.1); real activations would need trained weights,
so values are N(0,1) draws.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_LIB = os.path.join(_HERE, "libsynth_gen.so")
_lib = None

# tensor ids: one stream of random numbers per tensor
TID_K, TID_V, TID_LENS, TID_Q0 = 1, 2, 3, 16  # Q of layer l uses TID_Q0 + l


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.run(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC,
                        "-lm"], check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        u64 = ctypes.c_uint64
        lib.synth_raw_bits.argtypes = [u64, u64, u64]
        lib.synth_raw_bits.restype = u64
        lib.synth_normal_bf16.argtypes = [u64, u64, ctypes.c_double, u64, u64, ctypes.c_void_p]
        lib.synth_normal_bf16.restype = None
        _lib = lib
    return _lib


def normal_bf16(seed: int, tensor_id: int, count: int, mult: float = 1.0, first: int = 0,
                out: np.ndarray | None = None) -> np.ndarray:
    """bf16 bits of ``mult * N(0,1)`` for elements [first, first+count) of a tensor."""
    if out is None:
        out = np.empty(count, dtype=np.uint16)
    assert out.dtype == np.uint16 and out.size == count and out.flags.c_contiguous
    _load().synth_normal_bf16(seed, tensor_id, float(mult), first, count,
                              ctypes.c_void_p(out.ctypes.data))
    return out


def raw_bits(seed: int, tensor_id: int, counter: int) -> int:
    return int(_load().synth_raw_bits(seed, tensor_id, counter))


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = u + 0x7FFF + ((u >> 16) & 1)
    return (u >> 16).astype(np.uint16)


def e4m3_table() -> np.ndarray:
    """Values of the 256 FP8 E4M3 codes (1 sign, 4 exponent bits, bias 7, 3 mantissa bits; exponent
    field 0 subnormal; 0x7F / 0xFF NaN), float64."""
    code = np.arange(256)
    ex, man = (code >> 3) & 15, code & 7
    val = np.where(ex == 0, man / 8.0 * 2.0 ** -6, (1.0 + man / 8.0) * 2.0 ** (ex.astype(np.float64) - 7))
    val = np.where((ex == 15) & (man == 7), np.nan, val)
    return np.where(code >= 128, -val, val)


def quantize_e4m3(x: np.ndarray) -> np.ndarray:
    """Nearest E4M3 code of every element of x (float), ties to the even code, saturating at +-448."""
    pos = e4m3_table()[:127]                               # 0x00 .. 0x7E, ascending
    mid = (pos[:-1] + pos[1:]) / 2
    a = np.minimum(np.abs(np.asarray(x, dtype=np.float64)), 448.0)
    idx = np.searchsorted(mid, a, side="left")             # a == mid[i] -> i (the lower neighbour)
    tie = (idx < 126) & (a == mid[np.minimum(idx, 125)]) & (idx % 2 == 1)
    idx = idx + tie
    return (idx | np.where(np.signbit(x), 128, 0)).astype(np.uint8)


@dataclass
class Workload:
    """One seeded problem instance: shapes, lengths and the packed-layout offsets."""
    name: str
    B: int
    Hq: int
    Hkv: int
    d: int
    T: int
    layers: int
    seed: int
    kv_len: np.ndarray          # [B] int32, includes the T new positions
    k_mult: float = 1.0
    window: int = 0             # sliding window C (0 = plain causal)
    cu: np.ndarray = field(init=False)

    def __post_init__(self):
        self.kv_len = np.asarray(self.kv_len, dtype=np.int32)
        self.cu = np.zeros(self.B + 1, dtype=np.int32)
        np.cumsum(self.kv_len, out=self.cu[1:])

    @property
    def total_tokens(self) -> int:
        return int(self.cu[-1])

    @property
    def kv_elems(self) -> int:
        return self.total_tokens * self.Hkv * self.d

    @property
    def kv_bytes(self) -> int:
        """Algorithmic bytes of one layer call: every visible K and V element once."""
        return 2 * self.kv_elems * 2

    def make_q(self, layer: int) -> np.ndarray:
        return normal_bf16(self.seed, TID_Q0 + layer, self.B * self.Hq * self.T * self.d).reshape(
            self.B, self.Hq, self.T, self.d)

    def make_k(self) -> np.ndarray:
        return normal_bf16(self.seed, TID_K, self.kv_elems, mult=self.k_mult)

    def make_v(self) -> np.ndarray:
        return normal_bf16(self.seed, TID_V, self.kv_elems)

    def make_kv_fp8(self):
        """The same K and V draws stored as an 8-bit cache: (K8, V8, k_scale [Hkv], v_scale [Hkv]) with
        E4M3 bytes in the packed head-major layout and one scale per KV head, amax / 448 over all
        sequences, so that value = scale[c] * e4m3(byte)."""
        out = []
        all_bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
        with np.errstate(invalid="ignore"):
            all_vals = bf16_bits_to_f32(all_bits)            # every bf16 value, indexed by its bit pattern
        for make in (self.make_k, self.make_v):
            bits = make()
            amax = np.zeros(self.Hkv, dtype=np.float32)
            spans, off = [], 0                           # (head, first element, count) of every (sequence, head)
            for n in self.kv_len:
                per_head = int(n) * self.d
                for c in range(self.Hkv):
                    spans.append((c, off, per_head))
                    if per_head:                         # |x| grows with the low 15 bits of a finite bf16
                        top = int((bits[off:off + per_head] & 0x7FFF).max())
                        amax[c] = max(amax[c], float(all_vals[top]))
                    off += per_head
            scale = np.where(amax > 0, amax / 448.0, 1.0).astype(np.float32)
            # the quantiser is elementwise, so it is applied once to each of the 65,536 bf16 values per head
            # and then looked up: the same codes as quantising the tensor, at a fraction of the memory
            with np.errstate(invalid="ignore", over="ignore"):
                luts = [quantize_e4m3(np.nan_to_num(all_vals / scale[c], nan=0.0, posinf=448.0, neginf=-448.0))
                        for c in range(self.Hkv)]
            q = np.empty(bits.size, dtype=np.uint8)
            for c, first, count in spans:
                q[first:first + count] = luts[c][bits[first:first + count]]
            del bits
            out.append((q, scale))
        return out[0][0], out[1][0], out[0][1], out[1][1]


def ragged_lengths(seed: int, B: int, lo: int, span: int) -> np.ndarray:
    """N_i = lo + (draw_i mod span): seeded, not tile-aligned."""
    return np.array([lo + raw_bits(seed, TID_LENS, i) % span for i in range(B)], dtype=np.int32)


def workload(name: str) -> Workload:
    """The five benchmark configurations (plus scaled-down variants for quick tests)."""
    if name == "tiny":          # config 1
        return Workload(name, B=1, Hq=4, Hkv=1, d=64, T=1, layers=2, seed=0, kv_len=[512])
    if name == "3b_32k":        # config 2: keys scaled by 0.5 before rounding
        return Workload(name, B=1, Hq=32, Hkv=8, d=128, T=1, layers=13, seed=1, kv_len=[32768],
                        k_mult=0.5)
    if name == "ragged":        # config 3: N_i uniform in [4096, 131072]
        return Workload(name, B=16, Hq=32, Hkv=8, d=128, T=1, layers=1, seed=2,
                        kv_len=ragged_lengths(2, 16, 4096, 126977))
    if name == "1m":            # config 4
        return Workload(name, B=1, Hq=32, Hkv=8, d=128, T=1, layers=13, seed=3, kv_len=[1048576])
    if name == "128k":          # config 4's shape at 1/8 of the length (profiler captures)
        return Workload(name, B=1, Hq=32, Hkv=8, d=128, T=1, layers=13, seed=3, kv_len=[131072])
    if name == "chunk":         # config 5: 512 new rows appended after 262,144 cached keys
        return Workload(name, B=2, Hq=32, Hkv=8, d=128, T=512, layers=1, seed=4,
                        kv_len=[262144 + 512] * 2)
    if name == "chunk_32k":     # config 5 with a 32K cache (profiler captures)
        return Workload(name, B=2, Hq=32, Hkv=8, d=128, T=512, layers=1, seed=4,
                        kv_len=[32768 + 512] * 2)
    if name == "swa":           # batched decode under the paper's window of 1,024 (Section 4.1)
        return Workload(name, B=128, Hq=32, Hkv=8, d=128, T=1, layers=1, seed=6,
                        kv_len=ragged_lengths(6, 128, 2048, 2049), window=1024)
    if name == "ragged_small":  # same recipe as config 3, 32x shorter
        return Workload(name, B=16, Hq=32, Hkv=8, d=128, T=1, layers=1, seed=2,
                        kv_len=ragged_lengths(2, 16, 128, 3969))
    if name == "chunk_small":   # same recipe as config 5, shorter cache and chunk
        return Workload(name, B=2, Hq=32, Hkv=8, d=128, T=160, layers=1, seed=4,
                        kv_len=[1000 + 160, 777 + 160])
    raise KeyError(name)
