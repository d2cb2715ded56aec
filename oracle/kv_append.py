"""TEST INFRASTRUCTURE -- not part of the product.

fp64 oracle for the step that writes the shared cache (Section 2.2, first cross-decoder
equation):  K^ = LN(X) W_K,  V^ = LN(X) W_V,  with RMSNorm as LN and no bias (Section 2.1 /
Section 4.1: pre-RMSNorm, biases removed).  X holds the self-decoder's output for the T new
tokens of every sequence; the rows produced are appended to the head-major cache at positions
[N_i - T, N_i) of sequence i (kv_len counts them already, as in the attention calls).

Definition, written out (numpy fp64; the matrix product is the library's):

    r_t   = 1 / sqrt(mean_k x_{t,k}^2 + eps)
    y_t   = (x_t * r_t * g) @ W                     W = W_K or W_V, [d_model, Hkv * d]
    cache[i, c, N_i - T + t, :] = y_{i*T + t}[c*d : (c+1)*d]

Where the paper is silent: eps (1e-6 unless the caller says otherwise); the gain g multiplies
after the normalisation, as in the RMSNorm paper it cites.  Inputs are bf16 bit patterns
(uint16), converted exactly; nothing is rounded on the way.  Only tests, the smoke check and
the benchmark's CPU-baseline leg may import this module.
"""
from __future__ import annotations

import numpy as np


def _f64(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def rmsnorm_rows(X_bits, g_bits, eps: float = 1e-6) -> np.ndarray:
    """RMSNorm of every row of X [M, d_model] with gain g [d_model]; fp64."""
    X, g = _f64(X_bits), _f64(g_bits)
    r = 1.0 / np.sqrt((X * X).mean(axis=1, keepdims=True) + eps)
    return X * r * g


def kv_rows(X_bits, g_bits, Wk_bits, Wv_bits, eps: float = 1e-6):
    """(K^, V^) rows for the M tokens of X: two [M, Hkv*d] fp64 arrays."""
    Xn = rmsnorm_rows(X_bits, g_bits, eps)
    return Xn @ _f64(Wk_bits), Xn @ _f64(Wv_bits)


def append_positions(B: int, Hkv: int, d: int, T: int, cu, kv_len, kv_head_stride: int = 0) -> np.ndarray:
    """Element offset of cache row (i, c, N_i - T + t) for every token m = i*T + t and head c:
    int64 [B*T, Hkv], in the packed layout  cu[i]*Hkv*d + c*head_stride_i + j*d."""
    out = np.empty((B * T, Hkv), dtype=np.int64)
    for i in range(B):
        n = int(kv_len[i])
        if n < T:
            raise ValueError("kv_len must include the T new positions")
        hs = kv_head_stride if kv_head_stride else n * d
        for t in range(T):
            for c in range(Hkv):
                out[i * T + t, c] = int(cu[i]) * Hkv * d + c * hs + (n - T + t) * d
    return out


def kv_append(X_bits, g_bits, Wk_bits, Wv_bits, *, B, Hkv, d, T, cu, kv_len, eps=1e-6, kv_head_stride=0):
    """What the append must write: returns (offsets [B*T, Hkv], K_rows [B*T, Hkv, d], V_rows
    [B*T, Hkv, d]) -- the element offset of every new cache row and its fp64 contents."""
    Kr, Vr = kv_rows(X_bits, g_bits, Wk_bits, Wv_bits, eps)
    M = B * T
    if Kr.shape != (M, Hkv * d):
        raise ValueError("X must hold B*T rows and W must have Hkv*d columns")
    return (append_positions(B, Hkv, d, T, cu, kv_len, kv_head_stride),
            Kr.reshape(M, Hkv, d), Vr.reshape(M, Hkv, d))
