"""TEST INFRASTRUCTURE -- not part of the product.

ctypes front end of the fp64 CPU oracle (``xattn_oracle.c``) for the cross-decoder
attention over the shared K/V cache (Section 2.2 of the paper, cross-decoder
equations).  Only ``tests/``, ``__graft_entry__.smoke()`` and the CPU-baseline /
reference legs of ``bench.py`` may import this package; it imports nothing from
the CUDA package and the CUDA package never imports it.

All arrays are numpy.  Q, K, V are ``uint16`` arrays holding bf16 bit patterns
(the same bits the GPU reads); outputs are ``float64``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "xattn_oracle.c")
_LIB = os.path.join(_HERE, "liboracle_xattn.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, OpenMP parallel-for only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        i32, i64, f64, ptr = ctypes.c_int32, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        common = [i32, i32, i32, i32, i32, f64, ptr, ptr, ptr, ptr, ptr, i64, i32]
        lib.oracle_xattn.argtypes = common + [ptr, ptr]
        lib.oracle_xattn_rows.argtypes = common + [i64, ptr, ptr, ptr, ptr, ptr]
        lib.oracle_xattn_split_merge.argtypes = common + [i32, ptr, ptr, ptr]
        lib.oracle_combine.argtypes = [i64, i32, i32, ptr, ptr, ptr, ptr]
        lib.oracle_xattn_fp8.argtypes = [i32, i32, i32, i32, i32, f64, ptr, ptr, ptr, ptr, ptr, ptr, ptr, i64, i32,
                                         ptr, ptr]
        lib.oracle_xattn_fp8.restype = i32
        lib.oracle_e4m3_to_f64.argtypes = [ctypes.c_uint8]
        lib.oracle_e4m3_to_f64.restype = f64
        for f in (lib.oracle_xattn, lib.oracle_xattn_rows, lib.oracle_xattn_split_merge,
                  lib.oracle_combine, lib.oracle_num_threads):
            f.restype = i32
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _p(a: np.ndarray) -> ctypes.c_void_p:
    return ctypes.c_void_p(a.ctypes.data)


def _prep(Q, K, V, cu, kv_len, B, Hq, T, d):
    Q = np.ascontiguousarray(Q, dtype=np.uint16)
    K = np.ascontiguousarray(K, dtype=np.uint16).reshape(-1)
    V = np.ascontiguousarray(V, dtype=np.uint16).reshape(-1)
    cu = np.ascontiguousarray(cu, dtype=np.int32)
    kv_len = np.ascontiguousarray(kv_len, dtype=np.int32)
    if Q.size != B * Hq * T * d:
        raise ValueError("Q must hold B*Hq*T*d bf16 values")
    if cu.size != B + 1 or kv_len.size != B:
        raise ValueError("cu must have B+1 entries and kv_len B entries")
    return Q, K, V, cu, kv_len


def _check_extent(K, V, cu, kv_len, Hkv, d, kv_head_stride):
    need = 0
    for i in range(kv_len.size):
        hs = kv_head_stride if kv_head_stride else int(kv_len[i]) * d
        if kv_len[i] > 0:
            need = max(need, int(cu[i]) * Hkv * d + (Hkv - 1) * hs + int(kv_len[i]) * d)
    if K.size < need or V.size < need:
        raise ValueError("K/V buffers are smaller than the layout requires")


def xattn(Q, K, V, cu, kv_len, *, B, Hq, Hkv, d, T, scale=0.0, kv_head_stride=0, window=0):
    """Definition of the cross-attention; returns (O [B,Hq,T,d], LSE [B,Hq,T]) in fp64.
    ``window`` = C > 0 keeps, for the row at position i, only the keys i - C < j <= i (the
    sliding-window mask of Section 3.2); 0 = plain causal."""
    Q, K, V, cu, kv_len = _prep(Q, K, V, cu, kv_len, B, Hq, T, d)
    _check_extent(K, V, cu, kv_len, Hkv, d, kv_head_stride)
    O = np.empty((B, Hq, T, d), dtype=np.float64)
    LSE = np.empty((B, Hq, T), dtype=np.float64)
    rc = _load().oracle_xattn(B, Hq, Hkv, d, T, float(scale), _p(Q), _p(K), _p(V), _p(cu),
                              _p(kv_len), int(kv_head_stride), int(window), _p(O), _p(LSE))
    if rc:
        raise ValueError(f"oracle_xattn failed ({rc})")
    return O, LSE


def xattn_rows(Q, K, V, cu, kv_len, rows, *, B, Hq, Hkv, d, T, scale=0.0, kv_head_stride=0, window=0):
    """Same definition for selected rows; ``rows`` is an (n, 3) array of (b, h, t)."""
    Q, K, V, cu, kv_len = _prep(Q, K, V, cu, kv_len, B, Hq, T, d)
    _check_extent(K, V, cu, kv_len, Hkv, d, kv_head_stride)
    rows = np.asarray(rows, dtype=np.int32).reshape(-1, 3)
    rb = np.ascontiguousarray(rows[:, 0])
    rh = np.ascontiguousarray(rows[:, 1])
    rt = np.ascontiguousarray(rows[:, 2])
    n = rows.shape[0]
    O = np.empty((n, d), dtype=np.float64)
    LSE = np.empty((n,), dtype=np.float64)
    rc = _load().oracle_xattn_rows(B, Hq, Hkv, d, T, float(scale), _p(Q), _p(K), _p(V), _p(cu),
                                   _p(kv_len), int(kv_head_stride), int(window), n, _p(rb), _p(rh), _p(rt),
                                   _p(O), _p(LSE))
    if rc:
        raise ValueError(f"oracle_xattn_rows failed ({rc})")
    return O, LSE


def xattn_split_merge(Q, K, V, cu, kv_len, cuts, *, B, Hq, Hkv, d, T, scale=0.0, kv_head_stride=0, window=0):
    """The attention evaluated piecewise between the key positions ``cuts`` and merged by LSE."""
    Q, K, V, cu, kv_len = _prep(Q, K, V, cu, kv_len, B, Hq, T, d)
    _check_extent(K, V, cu, kv_len, Hkv, d, kv_head_stride)
    cuts = np.ascontiguousarray(cuts, dtype=np.int64)
    O = np.empty((B, Hq, T, d), dtype=np.float64)
    LSE = np.empty((B, Hq, T), dtype=np.float64)
    rc = _load().oracle_xattn_split_merge(B, Hq, Hkv, d, T, float(scale), _p(Q), _p(K), _p(V),
                                          _p(cu), _p(kv_len), int(kv_head_stride), int(window),
                                          int(cuts.size), _p(cuts), _p(O), _p(LSE))
    if rc:
        raise ValueError(f"oracle_xattn_split_merge failed ({rc})")
    return O, LSE


def combine(part_o, part_lse):
    """Merge partial results: part_o [rows,S,d] fp32, part_lse [rows,S] fp32 -> fp64 (O, LSE)."""
    part_o = np.ascontiguousarray(part_o, dtype=np.float32)
    part_lse = np.ascontiguousarray(part_lse, dtype=np.float32)
    rows, S, d = part_o.shape
    if part_lse.shape != (rows, S):
        raise ValueError("part_lse must be [rows, S]")
    O = np.empty((rows, d), dtype=np.float64)
    LSE = np.empty((rows,), dtype=np.float64)
    rc = _load().oracle_combine(rows, S, d, _p(part_o), _p(part_lse), _p(O), _p(LSE))
    if rc:
        raise ValueError(f"oracle_combine failed ({rc})")
    return O, LSE


def e4m3_to_f64(byte: int) -> float:
    """Value of one FP8 E4M3 byte (the oracle's own decoder)."""
    return float(_load().oracle_e4m3_to_f64(int(byte) & 0xFF))


def xattn_fp8(Q, K8, V8, k_scale, v_scale, cu, kv_len, *, B, Hq, Hkv, d, T, scale=0.0, kv_head_stride=0, window=0):
    """The same definition over an 8-bit cache: K8, V8 are uint8 E4M3 bytes in the packed head-major
    layout, k_scale / v_scale fp32 [Hkv]; an element's value is scale[c] * e4m3(byte)."""
    Q = np.ascontiguousarray(Q, dtype=np.uint16)
    K8 = np.ascontiguousarray(K8, dtype=np.uint8).reshape(-1)
    V8 = np.ascontiguousarray(V8, dtype=np.uint8).reshape(-1)
    k_scale = np.ascontiguousarray(k_scale, dtype=np.float32)
    v_scale = np.ascontiguousarray(v_scale, dtype=np.float32)
    cu = np.ascontiguousarray(cu, dtype=np.int32)
    kv_len = np.ascontiguousarray(kv_len, dtype=np.int32)
    if Q.size != B * Hq * T * d or k_scale.size != Hkv or v_scale.size != Hkv:
        raise ValueError("Q must hold B*Hq*T*d values and the scales Hkv values each")
    _check_extent(K8, V8, cu, kv_len, Hkv, d, kv_head_stride)
    O = np.empty((B, Hq, T, d), dtype=np.float64)
    LSE = np.empty((B, Hq, T), dtype=np.float64)
    rc = _load().oracle_xattn_fp8(B, Hq, Hkv, d, T, float(scale), _p(Q), _p(K8), _p(V8), _p(k_scale), _p(v_scale),
                                  _p(cu), _p(kv_len), int(kv_head_stride), int(window), _p(O), _p(LSE))
    if rc:
        raise ValueError(f"oracle_xattn_fp8 failed ({rc})")
    return O, LSE

