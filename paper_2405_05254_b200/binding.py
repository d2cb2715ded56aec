"""Thin ctypes binding of the C-ABI library (argument marshalling only).

Function names mirror ``include/yoco_xattn.h``.  Tensors are torch CUDA tensors (torch is used
for device memory and streams only); lengths and offsets are host numpy int32 arrays.  There is
no fallback: if the CUDA library has not been built, every call raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libyoco_xattn.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE_TOO_SMALL, ERR_CUDA, ERR_TIMEOUT = 0, -1, -2, -3, -4, -5
ERR_STATIC_SCRATCH_EXCEEDED = -6
MODE_DECODE, MODE_CHUNK = 0, 1


class Shape(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("Hq", ctypes.c_int32), ("Hkv", ctypes.c_int32),
                ("d", ctypes.c_int32), ("T", ctypes.c_int32), ("scale", ctypes.c_float),
                ("kv_head_stride", ctypes.c_int64), ("max_kv_len", ctypes.c_int32),
                ("window", ctypes.c_int32)]


class KvAppendShape(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("Hkv", ctypes.c_int32), ("d", ctypes.c_int32), ("T", ctypes.c_int32),
                ("d_model", ctypes.c_int32), ("eps", ctypes.c_float), ("kv_head_stride", ctypes.c_int64)]


class Segment(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("group", "b", "c", "k_begin", "k_end", "slot")]


class PlanInfo(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("mode", "tile_n", "tile_m", "m_tiles", "num_groups", "num_ctas", "num_streams",
                 "num_segments", "max_splits", "needs_combine")] + \
               [("total_tiles", ctypes.c_int64), ("workspace_bytes", ctypes.c_int64),
                ("sub_items", ctypes.c_int32), ("num_slots", ctypes.c_int32)]


class YocoError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().yoco_xattn_strerror(code).decode()
        if code == ERR_CUDA:
            msg += f" [cudaError {lib().yoco_xattn_last_cuda_error()}]"
        super().__init__(f"{where}: {msg} ({code})")


_lib = None


def lib() -> ctypes.CDLL:
    """Load libyoco_xattn.so; fails loudly when it is missing (there is no CPU path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with paper_2405_05254_b200.build.build_cuda_library()")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
        L.yoco_xattn_plan.argtypes = [ctypes.POINTER(Shape), vp, i32, i32, ctypes.POINTER(PlanInfo), vp, i32]
        L.yoco_xattn_workspace_size.argtypes = [ctypes.POINTER(Shape), vp, i32, i32, ctypes.POINTER(sz)]
        run_args = [ctypes.POINTER(Shape), vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.yoco_xattn_decode.argtypes = run_args
        L.yoco_xattn_chunk.argtypes = run_args
        L.yoco_xattn_decode_static.argtypes = [ctypes.POINTER(Shape), vp, vp, vp, vp, vp, vp, vp, vp]
        L.yoco_xattn_static_scratch_bytes.argtypes = []
        L.yoco_xattn_combine.argtypes = [i64, i32, i32, vp, vp, vp, vp, vp]
        L.yoco_xattn_combine_gathered.argtypes = [i64, i32, i32, vp, vp, vp, vp, vp]
        L.yoco_xattn_decode_partial.argtypes = [ctypes.POINTER(Shape), vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        part_at = [ctypes.POINTER(Shape), vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.yoco_xattn_decode_partial_at.argtypes = part_at
        L.yoco_xattn_chunk_partial_at.argtypes = part_at
        L.yoco_xattn_workspace_size_at.argtypes = [ctypes.POINTER(Shape), vp, vp, vp, i32, i32, ctypes.POINTER(sz)]
        L.yoco_xattn_plan_at.argtypes = [ctypes.POINTER(Shape), vp, vp, vp, i32, i32, ctypes.POINTER(PlanInfo), vp, i32]
        for name in ("yoco_xattn_decode_partial_at", "yoco_xattn_chunk_partial_at", "yoco_xattn_workspace_size_at",
                     "yoco_xattn_plan_at"):
            getattr(L, name).restype = i32
        L.yoco_xattn_decode_fp8.argtypes = [ctypes.POINTER(Shape), vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.yoco_xattn_decode_fp8.restype = i32
        L.yoco_xattn_chunk_fp8.argtypes = L.yoco_xattn_decode_fp8.argtypes
        L.yoco_xattn_chunk_fp8.restype = i32
        L.yoco_xattn_workspace_size_chunk_fp8.argtypes = [ctypes.POINTER(Shape), vp, i32, ctypes.POINTER(sz)]
        L.yoco_xattn_workspace_size_chunk_fp8.restype = i32
        L.yoco_kv_fold_gain.argtypes = [i64, i64, vp, vp, vp, vp]
        L.yoco_kv_append.argtypes = [ctypes.POINTER(KvAppendShape), vp, vp, vp, vp, vp, vp, vp, vp]
        L.yoco_xattn_sub_bound.argtypes = [ctypes.c_int64, i32, i32]
        L.yoco_xattn_sub_bound.restype = ctypes.c_int64
        L.yoco_kv_append_fp8.argtypes = [ctypes.POINTER(KvAppendShape), vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.yoco_kv_append_fp8.restype = i32
        L.yoco_kv_append_status.argtypes = [vp]
        for name in ("yoco_kv_fold_gain", "yoco_kv_append", "yoco_kv_append_status"):
            getattr(L, name).restype = i32
        L.yoco_xattn_status.argtypes = [vp, vp]
        L.yoco_xattn_status_detail.argtypes = [vp, vp, ctypes.POINTER(i32), ctypes.POINTER(i32)]
        L.yoco_xattn_decode_status_word.argtypes = [i32, ctypes.POINTER(i32), ctypes.POINTER(i32)]
        L.yoco_kv_append_status_detail.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(i32)]
        L.yoco_xattn_selftest_wait_expiry.argtypes = [ctypes.POINTER(Shape), vp, vp, vp, vp, vp, vp, vp, sz, i32, vp]
        for name in ("yoco_xattn_status_detail", "yoco_xattn_decode_status_word", "yoco_kv_append_status_detail",
                     "yoco_xattn_selftest_wait_expiry"):
            getattr(L, name).restype = i32
        L.yoco_xattn_profile_enable.argtypes = [i32]
        L.yoco_xattn_profile_collect.argtypes = [vp, i32, vp]
        L.yoco_xattn_strerror.argtypes = [i32]
        L.yoco_xattn_strerror.restype = ctypes.c_char_p
        L.yoco_xattn_last_cuda_error.argtypes = []
        for name in ("plan", "workspace_size", "decode", "chunk", "combine", "status", "last_cuda_error",
                     "profile_enable", "profile_collect", "decode_static", "static_scratch_bytes",
                     "combine_gathered", "decode_partial"):
            getattr(L, "yoco_xattn_" + name).restype = i32
        _lib = L
    return _lib


def make_shape(B, Hq, Hkv, d, T, scale=0.0, kv_head_stride=0, max_kv_len=0, window=0) -> Shape:
    """``window`` = C > 0 selects the sliding-window mask (row i sees i - C < j <= i); 0 = none."""
    return Shape(B, Hq, Hkv, d, T, float(scale), int(kv_head_stride), int(max_kv_len), int(window))


def _host_i32(a):
    if a is None:
        return None, None
    arr = np.ascontiguousarray(a, dtype=np.int32)
    return arr, ctypes.c_void_p(arr.ctypes.data)


def yoco_xattn_plan(shape: Shape, kv_len, sm_count: int, mode: int):
    """Returns (PlanInfo, list of Segment) of the split/tile heuristic; host only."""
    keep, p_len = _host_i32(kv_len)
    info = PlanInfo()
    rc = lib().yoco_xattn_plan(ctypes.byref(shape), p_len, sm_count, mode, ctypes.byref(info), None, 0)
    if rc != OK:
        raise YocoError(rc, "yoco_xattn_plan")
    segs = (Segment * max(1, info.num_segments))()
    rc = lib().yoco_xattn_plan(ctypes.byref(shape), p_len, sm_count, mode, ctypes.byref(info),
                               ctypes.cast(segs, ctypes.c_void_p), info.num_segments)
    if rc != OK:
        raise YocoError(rc, "yoco_xattn_plan")
    return info, list(segs)[: info.num_segments]


def yoco_xattn_plan_at(shape: Shape, kv_len, key_offset, kv_total, sm_count: int, mode: int):
    """(PlanInfo, segments) for one key shard at a given place in the whole sequences; host only."""
    keep, p_len = _host_i32(kv_len)
    keep_off, p_off = _host_i32(key_offset)
    keep_tot, p_tot = _host_i32(kv_total)
    info = PlanInfo()
    rc = lib().yoco_xattn_plan_at(ctypes.byref(shape), p_len, p_off, p_tot, sm_count, mode, ctypes.byref(info), None, 0)
    if rc != OK:
        raise YocoError(rc, "yoco_xattn_plan_at")
    segs = (Segment * max(1, info.num_segments))()
    rc = lib().yoco_xattn_plan_at(ctypes.byref(shape), p_len, p_off, p_tot, sm_count, mode, ctypes.byref(info),
                                  ctypes.cast(segs, ctypes.c_void_p), info.num_segments)
    if rc != OK:
        raise YocoError(rc, "yoco_xattn_plan_at")
    return info, list(segs)[: info.num_segments]


def yoco_xattn_workspace_size(shape: Shape, kv_len, mode: int, sm_count: int = 0) -> int:
    keep, p_len = _host_i32(kv_len)
    out = ctypes.c_size_t(0)
    rc = lib().yoco_xattn_workspace_size(ctypes.byref(shape), p_len, sm_count, mode, ctypes.byref(out))
    if rc != OK:
        raise YocoError(rc, "yoco_xattn_workspace_size")
    return int(out.value)


def _ptr(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else None


def _stream_ptr(stream):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _run(fn_name, shape, Q, K, V, cu_kv, kv_len, O, lse, workspace, stream):
    keep_cu, p_cu = _host_i32(cu_kv)
    keep_len, p_len = _host_i32(kv_len)
    fn = getattr(lib(), fn_name)
    rc = fn(ctypes.byref(shape), _ptr(Q), _ptr(K), _ptr(V), p_cu, p_len, _ptr(O), _ptr(lse),
            _ptr(workspace), workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    if rc != OK:
        raise YocoError(rc, fn_name)


def yoco_xattn_decode(shape: Shape, Q, K, V, cu_kv, kv_len, O, lse, workspace, stream=None) -> None:
    """Enqueue split-KV decode attention (G*T <= 16 rows per KV head) on the stream."""
    _run("yoco_xattn_decode", shape, Q, K, V, cu_kv, kv_len, O, lse, workspace, stream)


class PreparedCall:
    """A decode or chunk call whose arguments are marshalled once: a serving loop that makes the same
    layer call every step (same buffers, same lengths) pays the ctypes conversions a single time.
    The tensors and arrays are kept alive by the object; run() only enqueues."""

    def __init__(self, fn_name, shape, Q, K, V, cu_kv, kv_len, O, lse, workspace, stream=None):
        self._keep = (shape, Q, K, V, O, lse, workspace, stream) + _host_i32(cu_kv)[:1] + _host_i32(kv_len)[:1]
        p_cu = None if self._keep[-2] is None else ctypes.c_void_p(self._keep[-2].ctypes.data)
        p_len = None if self._keep[-1] is None else ctypes.c_void_p(self._keep[-1].ctypes.data)
        self._name = fn_name
        self._fn = getattr(lib(), fn_name)
        self._args = (ctypes.byref(shape), _ptr(Q), _ptr(K), _ptr(V), p_cu, p_len, _ptr(O), _ptr(lse), _ptr(workspace),
                      ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream_ptr(stream))

    def run(self) -> None:
        rc = self._fn(*self._args)
        if rc != OK:
            raise YocoError(rc, self._name)


def prepare_decode(shape: Shape, Q, K, V, cu_kv, kv_len, O, lse, workspace, stream=None) -> PreparedCall:
    """yoco_xattn_decode with its arguments marshalled once; call .run() to enqueue it."""
    return PreparedCall("yoco_xattn_decode", shape, Q, K, V, cu_kv, kv_len, O, lse, workspace, stream)


def yoco_xattn_chunk(shape: Shape, Q, K, V, cu_kv, kv_len, O, lse, workspace, stream=None) -> None:
    """Enqueue the multi-token (tcgen05) attention on the stream."""
    _run("yoco_xattn_chunk", shape, Q, K, V, cu_kv, kv_len, O, lse, workspace, stream)


def yoco_xattn_combine(part_o, part_lse, O, lse=None, stream=None) -> None:
    """Merge partials: part_o [rows,S,d] fp32, part_lse [rows,S] fp32 -> O [rows,d] bf16."""
    rows, S, d = part_o.shape
    rc = lib().yoco_xattn_combine(rows, S, d, _ptr(part_o), _ptr(part_lse), _ptr(O), _ptr(lse),
                                  _stream_ptr(stream))
    if rc != OK:
        raise YocoError(rc, "yoco_xattn_combine")


def yoco_xattn_combine_gathered(part_o, part_lse, O, lse=None, stream=None) -> None:
    """Merge piece-major partials: part_o [S,rows,d] fp32, part_lse [S,rows] fp32 -> O [rows,d] bf16."""
    S, rows, d = part_o.shape
    rc = lib().yoco_xattn_combine_gathered(rows, S, d, _ptr(part_o), _ptr(part_lse), _ptr(O), _ptr(lse),
                                           _stream_ptr(stream))
    if rc != OK:
        raise YocoError(rc, "yoco_xattn_combine_gathered")


def yoco_xattn_decode_partial(shape: Shape, Q, K, V, cu_kv, kv_len, part_o, part_lse, workspace,
                              stream=None) -> None:
    """Decode over the key shard this GPU holds: fp32 partial rows + their log-sum-exp (T = 1)."""
    keep_cu, p_cu = _host_i32(cu_kv)
    keep_len, p_len = _host_i32(kv_len)
    rc = lib().yoco_xattn_decode_partial(ctypes.byref(shape), _ptr(Q), _ptr(K), _ptr(V), p_cu, p_len,
                                         _ptr(part_o), _ptr(part_lse), _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    if rc != OK:
        raise YocoError(rc, "yoco_xattn_decode_partial")


def yoco_xattn_partial_at(shape: Shape, Q, K, V, cu_kv, kv_len, key_offset, kv_total, part_o, part_lse, workspace,
                          mode: int = MODE_DECODE, stream=None) -> None:
    """One key shard's partial result with the shard's place in the whole sequences (host int32 [B] each:
    first key held here, length of the whole sequence): any T and any window.  ``mode`` picks the split-KV
    decode kernel (G*T <= 16) or the tensor-core chunk kernel."""
    keep_cu, p_cu = _host_i32(cu_kv)
    keep_len, p_len = _host_i32(kv_len)
    keep_off, p_off = _host_i32(key_offset)
    keep_tot, p_tot = _host_i32(kv_total)
    name = "yoco_xattn_decode_partial_at" if mode == MODE_DECODE else "yoco_xattn_chunk_partial_at"
    rc = getattr(lib(), name)(ctypes.byref(shape), _ptr(Q), _ptr(K), _ptr(V), p_cu, p_len, p_off, p_tot,
                              _ptr(part_o), _ptr(part_lse), _ptr(workspace),
                              workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    if rc != OK:
        raise YocoError(rc, name)


def yoco_xattn_workspace_size_at(shape: Shape, kv_len, key_offset, kv_total, mode: int, sm_count: int = 0) -> int:
    keep_len, p_len = _host_i32(kv_len)
    keep_off, p_off = _host_i32(key_offset)
    keep_tot, p_tot = _host_i32(kv_total)
    out = ctypes.c_size_t(0)
    rc = lib().yoco_xattn_workspace_size_at(ctypes.byref(shape), p_len, p_off, p_tot, sm_count, mode, ctypes.byref(out))
    if rc != OK:
        raise YocoError(rc, "yoco_xattn_workspace_size_at")
    return int(out.value)


def yoco_xattn_decode_fp8(shape: Shape, Q, K8, V8, k_scale, v_scale, cu_kv, kv_len, O, lse, workspace,
                          stream=None) -> None:
    """Decode over an FP8 E4M3 cache (uint8 device tensors) with per-head scales (host float32 [Hkv])."""
    keep_cu, p_cu = _host_i32(cu_kv)
    keep_len, p_len = _host_i32(kv_len)
    ks = np.ascontiguousarray(k_scale, dtype=np.float32)
    vs = np.ascontiguousarray(v_scale, dtype=np.float32)
    rc = lib().yoco_xattn_decode_fp8(ctypes.byref(shape), _ptr(Q), _ptr(K8), _ptr(V8),
                                     ctypes.c_void_p(ks.ctypes.data), ctypes.c_void_p(vs.ctypes.data), p_cu, p_len,
                                     _ptr(O), _ptr(lse), _ptr(workspace),
                                     workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    if rc != OK:
        raise YocoError(rc, "yoco_xattn_decode_fp8")


def yoco_xattn_chunk_fp8(shape: Shape, Q, K8, V8, k_scale, v_scale, cu_kv, kv_len, O, lse, workspace,
                         stream=None) -> None:
    """The multi-token (tensor-core) path over an FP8 E4M3 cache with per-head scales; any T."""
    keep_cu, p_cu = _host_i32(cu_kv)
    keep_len, p_len = _host_i32(kv_len)
    ks = np.ascontiguousarray(k_scale, dtype=np.float32)
    vs = np.ascontiguousarray(v_scale, dtype=np.float32)
    rc = lib().yoco_xattn_chunk_fp8(ctypes.byref(shape), _ptr(Q), _ptr(K8), _ptr(V8),
                                    ctypes.c_void_p(ks.ctypes.data), ctypes.c_void_p(vs.ctypes.data), p_cu, p_len,
                                    _ptr(O), _ptr(lse), _ptr(workspace),
                                    workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    if rc != OK:
        raise YocoError(rc, "yoco_xattn_chunk_fp8")


def yoco_xattn_workspace_size_chunk_fp8(shape: Shape, kv_len, sm_count: int = 0) -> int:
    keep, p_len = _host_i32(kv_len)
    out = ctypes.c_size_t(0)
    rc = lib().yoco_xattn_workspace_size_chunk_fp8(ctypes.byref(shape), p_len, sm_count, ctypes.byref(out))
    if rc != OK:
        raise YocoError(rc, "yoco_xattn_workspace_size_chunk_fp8")
    return int(out.value)


def yoco_kv_fold_gain(g, W, Wg, stream=None) -> None:
    """Wg = g[:, None] * W rounded to bf16 (W, Wg: [d_model, n_out] bf16 device tensors)."""
    d_model, n_out = W.shape
    rc = lib().yoco_kv_fold_gain(d_model, n_out, _ptr(g), _ptr(W), _ptr(Wg), _stream_ptr(stream))
    if rc != OK:
        raise YocoError(rc, "yoco_kv_fold_gain")


def yoco_kv_append(shape: KvAppendShape, X, Wgk, Wgv, K, V, cu_kv, kv_len, stream=None) -> None:
    """Enqueue K^ = RMSNorm(X) W_K, V^ = RMSNorm(X) W_V and store the rows at the last T positions
    of every sequence in the packed caches K, V (in place)."""
    keep_cu, p_cu = _host_i32(cu_kv)
    keep_len, p_len = _host_i32(kv_len)
    rc = lib().yoco_kv_append(ctypes.byref(shape), _ptr(X), _ptr(Wgk), _ptr(Wgv), _ptr(K), _ptr(V), p_cu, p_len,
                              _stream_ptr(stream))
    if rc != OK:
        raise YocoError(rc, "yoco_kv_append")


def yoco_xattn_sub_bound(n_tiles: int, sub_items: int, r: int) -> int:
    return int(lib().yoco_xattn_sub_bound(n_tiles, sub_items, r))


def yoco_kv_append_fp8(shape: KvAppendShape, X, Wgk, Wgv, K8, V8, k_scale, v_scale, cu_kv, kv_len, stream=None) -> None:
    """As yoco_kv_append, but the rows are stored as FP8 E4M3 bytes (uint8 caches) after division by the
    per-head scales (host float32 [Hkv])."""
    keep_cu, p_cu = _host_i32(cu_kv)
    keep_len, p_len = _host_i32(kv_len)
    ks = np.ascontiguousarray(k_scale, dtype=np.float32)
    vs = np.ascontiguousarray(v_scale, dtype=np.float32)
    rc = lib().yoco_kv_append_fp8(ctypes.byref(shape), _ptr(X), _ptr(Wgk), _ptr(Wgv), _ptr(K8), _ptr(V8),
                                  ctypes.c_void_p(ks.ctypes.data), ctypes.c_void_p(vs.ctypes.data), p_cu, p_len,
                                  _stream_ptr(stream))
    if rc != OK:
        raise YocoError(rc, "yoco_kv_append_fp8")


def yoco_kv_append_status(stream=None) -> int:
    """Synchronise the stream; 0 unless an append kernel gave up a bounded wait since the last call."""
    return int(lib().yoco_kv_append_status(_stream_ptr(stream)))


def yoco_xattn_status(workspace, stream=None) -> int:
    """Synchronise the stream and return the status of the last call that used ``workspace`` (0 = ok);
    ``workspace=None`` reads the built-in buffer of yoco_xattn_decode_static on the current device."""
    return int(lib().yoco_xattn_status(_ptr(workspace), _stream_ptr(stream)))


WAIT_ITEM_QUEUE, WAIT_RING_FULL, WAIT_RING_EMPTY, WAIT_TENSOR, WAIT_DRAIN, WAIT_MISALIGNED = 1, 2, 3, 4, 5, 6


def yoco_xattn_status_detail(workspace, stream=None):
    """(status, wait_class, cta): which kind of bounded wait ran out first, and in which CTA."""
    wc, cta = ctypes.c_int32(0), ctypes.c_int32(0)
    rc = lib().yoco_xattn_status_detail(_ptr(workspace), _stream_ptr(stream), ctypes.byref(wc), ctypes.byref(cta))
    return int(rc), int(wc.value), int(cta.value)


def yoco_xattn_decode_status_word(word: int):
    """Pure host: (status, wait_class, cta) of a status word."""
    wc, cta = ctypes.c_int32(0), ctypes.c_int32(0)
    rc = lib().yoco_xattn_decode_status_word(int(word), ctypes.byref(wc), ctypes.byref(cta))
    return int(rc), int(wc.value), int(cta.value)


def yoco_kv_append_status_detail(stream=None):
    wc, cta = ctypes.c_int32(0), ctypes.c_int32(0)
    rc = lib().yoco_kv_append_status_detail(_stream_ptr(stream), ctypes.byref(wc), ctypes.byref(cta))
    return int(rc), int(wc.value), int(cta.value)


def yoco_xattn_selftest_wait_expiry(shape: Shape, Q, K, V, cu_kv, kv_len, O, workspace, limit_ms: int, stream=None) -> None:
    """Run the decode kernel with a producer that starts no copy and a wait limit of ``limit_ms``: the
    first tile wait runs out, the kernel records it and returns.  O is left undefined."""
    keep_cu, p_cu = _host_i32(cu_kv)
    keep_len, p_len = _host_i32(kv_len)
    rc = lib().yoco_xattn_selftest_wait_expiry(ctypes.byref(shape), _ptr(Q), _ptr(K), _ptr(V), p_cu, p_len, _ptr(O),
                                               _ptr(workspace), workspace.numel() * workspace.element_size(),
                                               int(limit_ms), _stream_ptr(stream))
    if rc != OK:
        raise YocoError(rc, "yoco_xattn_selftest_wait_expiry")


def yoco_xattn_selftest_wait_expiry_fp8(shape: Shape, Q, K8, V8, k_scale, v_scale, cu_kv, kv_len, O, workspace,
                                        limit_ms: int, stream=None) -> None:
    """The same self-test for the decode kernel of the 8-bit cache: the wait that runs out is the consumers'
    wait for the producer to arm their tile.  O is left undefined."""
    keep_cu, p_cu = _host_i32(cu_kv)
    keep_len, p_len = _host_i32(kv_len)
    ks = np.ascontiguousarray(k_scale, dtype=np.float32)
    vs = np.ascontiguousarray(v_scale, dtype=np.float32)
    rc = lib().yoco_xattn_selftest_wait_expiry_fp8(ctypes.byref(shape), _ptr(Q), _ptr(K8), _ptr(V8),
                                                   ctypes.c_void_p(ks.ctypes.data), ctypes.c_void_p(vs.ctypes.data),
                                                   p_cu, p_len, _ptr(O), _ptr(workspace),
                                                   workspace.numel() * workspace.element_size(), int(limit_ms),
                                                   _stream_ptr(stream))
    if rc != OK:
        raise YocoError(rc, "yoco_xattn_selftest_wait_expiry_fp8")


def yoco_xattn_profile_enable(max_records: int) -> None:
    rc = lib().yoco_xattn_profile_enable(max_records)
    if rc != OK:
        raise YocoError(rc, "yoco_xattn_profile_enable")


def yoco_xattn_profile_collect(capacity: int) -> np.ndarray:
    """Durations (ms) of the attention kernel of the calls recorded since the last collect."""
    buf = np.zeros(max(1, capacity), dtype=np.float32)
    n = ctypes.c_int32(0)
    rc = lib().yoco_xattn_profile_collect(ctypes.c_void_p(buf.ctypes.data), capacity, ctypes.byref(n))
    if rc != OK:
        raise YocoError(rc, "yoco_xattn_profile_collect")
    return buf[: n.value].copy()


def yoco_xattn_decode_static(shape: Shape, Q, K, V, cu_kv, kv_len, O, lse, stream=None) -> None:
    """Decode for callers that cannot allocate: same result as yoco_xattn_decode, but the split
    tables and partial results live in a 4 MiB buffer built into the library instead of a
    caller-provided workspace.  Raises YocoError(ERR_STATIC_SCRATCH_EXCEEDED) when the problem
    needs more than that.  Calls that may overlap on the GPU must not both use this entry."""
    keep_cu, p_cu = _host_i32(cu_kv)
    keep_len, p_len = _host_i32(kv_len)
    rc = lib().yoco_xattn_decode_static(ctypes.byref(shape), _ptr(Q), _ptr(K), _ptr(V), p_cu, p_len,
                                        _ptr(O), _ptr(lse), _stream_ptr(stream))
    if rc != OK:
        raise YocoError(rc, "yoco_xattn_decode_static")


def yoco_xattn_static_scratch_bytes() -> int:
    return int(lib().yoco_xattn_static_scratch_bytes())
