"""TEST INFRASTRUCTURE -- how far an 8-bit (FP8 E4M3) K/V cache moves the attention output.

Section 1 of the paper sizes a cache under 8-bit K/V quantisation and says nothing about its
accuracy.  This script measures, with the fp64 oracle only (no GPU, nothing from the CUDA package),
the distance between the attention over a bf16 cache and over the same cache rounded to E4M3 with
per-head scales, for the decode shape of the benchmark (B = 1, 32 query heads over 8 KV heads,
d = 128, T = 1) at N = 32K, 128K and 1M keys, for two score distributions and three scale choices:

  scores   gaussian: q, k ~ N(0, 1), score standard deviation 1 (in units of 1/sqrt(d) q.k)
           peaked:   keys scaled by 4, score standard deviation 4: a handful of keys carry the weight
  scale    amax/448:      the largest magnitude of the head maps to the largest E4M3 value (no clipping)
           4*amax/448:    the same with two bits of range thrown away (more values land on subnormals)
           3 sigma/448:   values beyond three standard deviations saturate (0.27 % of a Gaussian)

Usage:  python -m oracle.fp8_tolerance_study [--max-keys 1048576]      (prints a Markdown table)
"""
from __future__ import annotations

import argparse
import sys
import time

import numpy as np

import oracle
import synth_inputs as si


def quantise(bits: np.ndarray, Hkv: int, N: int, d: int, scale: np.ndarray) -> np.ndarray:
    """E4M3 codes of a [Hkv, N, d] bf16 tensor divided by per-head scales (nearest even, saturating)."""
    all_vals = si.bf16_bits_to_f32(np.arange(65536, dtype=np.uint32).astype(np.uint16))
    out = np.empty(bits.size, dtype=np.uint8)
    per_head = N * d
    for c in range(Hkv):
        with np.errstate(invalid="ignore", over="ignore"):
            lut = si.quantize_e4m3(np.nan_to_num(all_vals / scale[c], nan=0.0, posinf=448.0, neginf=-448.0))
        out[c * per_head:(c + 1) * per_head] = lut[bits[c * per_head:(c + 1) * per_head]]
    return out


def head_stats(bits: np.ndarray, Hkv: int, N: int, d: int):
    """Per-head largest magnitude and standard deviation of a [Hkv, N, d] bf16 tensor."""
    amax, sigma = np.zeros(Hkv), np.zeros(Hkv)
    for c in range(Hkv):
        x = si.bf16_bits_to_f32(bits[c * N * d:(c + 1) * N * d])
        amax[c] = float(np.abs(x).max())
        sigma[c] = float(np.sqrt(np.mean(x.astype(np.float64) ** 2)))
    return amax, sigma


def study(max_keys: int):
    B, Hq, Hkv, d, T = 1, 32, 8, 128, 1
    rows = []
    for N in (32768, 131072, 1048576):
        if N > max_keys:
            continue
        for name, k_mult in (("gaussian", 1.0), ("peaked", 4.0)):
            w = si.Workload(f"fp8_study_{name}", B=B, Hq=Hq, Hkv=Hkv, d=d, T=T, layers=1, seed=77, kv_len=[N], k_mult=k_mult)
            K, V, Q = w.make_k(), w.make_v(), w.make_q(0)
            kw = dict(B=B, Hq=Hq, Hkv=Hkv, d=d, T=T)
            o_ref, lse_ref = oracle.xattn(Q, K, V, w.cu, w.kv_len, **kw)
            ka, ks = head_stats(K, Hkv, N, d)
            va, vs = head_stats(V, Hkv, N, d)
            for label, k_scale, v_scale in (("amax/448", ka / 448, va / 448),
                                            ("4*amax/448", 4 * ka / 448, 4 * va / 448),
                                            ("3 sigma/448", 3 * ks / 448, 3 * vs / 448)):
                k_scale, v_scale = k_scale.astype(np.float32), v_scale.astype(np.float32)
                K8, V8 = quantise(K, Hkv, N, d, k_scale), quantise(V, Hkv, N, d, v_scale)
                o8, lse8 = oracle.xattn_fp8(Q, K8, V8, k_scale, v_scale, w.cu, w.kv_len, **kw)
                diff = o8 - o_ref
                rows.append((N, name, label, float(np.linalg.norm(diff) / np.linalg.norm(o_ref)),
                             float(np.abs(diff).max()), float(np.abs(o_ref).max()), float(np.abs(lse8 - lse_ref).max())))
                print(f"# N={N} {name} {label}: rel-L2 {rows[-1][3]:.3e}", file=sys.stderr, flush=True)
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--max-keys", type=int, default=1048576)
    args = ap.parse_args()
    t0 = time.time()
    rows = study(args.max_keys)
    print("| keys | scores | scale | rel-L2 of O (fp8 cache vs bf16 cache) | max abs diff | max abs O | max abs LSE diff |")
    print("|---|---|---|---|---|---|---|")
    for N, name, label, rel, mx, omax, dl in rows:
        print(f"| {N:,} | {name} | {label} | {rel:.2e} | {mx:.2e} | {omax:.2e} | {dl:.2e} |")
    print(f"\n(oracle only, fp64; {time.time() - t0:.0f} s on {oracle.num_threads()} threads)")


if __name__ == "__main__":
    main()
