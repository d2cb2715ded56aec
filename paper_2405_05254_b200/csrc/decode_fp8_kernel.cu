// Split-KV decode over an 8-bit cache: K and V stored as FP8 E4M3 bytes with one fp32 scale per
// KV head (value = scale[c] * e4m3(byte)), head dimension 128.  Same structure as the bf16 decode
// kernel (one CTA per contiguous range of the flat (stream, key tile) space, a TMA producer warp,
// four consumer warps with their own online-softmax state), but a 64-key tile is 8 KB per tensor,
// so the same HBM bandwidth streams twice as many keys, and each consumer warp takes whole tiles
// in turn (instead of a quarter of every tile) so that its fixed latencies are paid per 64 keys.
//
// The bytes are widened to fp16 in registers (cvt.rn.f16x2.e4m3x2 is exact) and the small
// products run as m16n8k16 fp16 MMAs with fp32 accumulation; Q is converted bf16 -> fp16 once per
// segment and P is rounded to fp16.  Because ldmatrix moves 16-bit units, a lane receives four
// consecutive channels of a key (K) or two channels of two consecutive keys (V, transposed); the
// reduction index of an MMA may be permuted freely as long as both operands agree, so Q is loaded
// with the matching channel order and the output channels are put back in order when the
// accumulators are written out.  The scales multiply the scores (k_scale, folded into the softmax
// scale) and the output (v_scale).
#include <cuda_fp16.h>

#include "kernels.h"
#include "ptx.cuh"

namespace yoco {

namespace {

constexpr int kConsumerWarps = 4;
constexpr int kThreads = (kConsumerWarps + 1) * 32;
constexpr int TILE_N = kDecodeTileN;          // 64 keys
constexpr int D = 128;                        // head dimension = bytes per key row
constexpr int TENSOR_BYTES = TILE_N * D;      // 8 KB: 64 rows x 128 B, 128-byte swizzle
constexpr int STAGE_BYTES = 2 * TENSOR_BYTES;

template <int ROWS>
struct Cfg8 {
    static constexpr int MERGE_O_BYTES = kConsumerWarps * ROWS * D * 4;
    static constexpr int MERGE_ML_BYTES = kConsumerWarps * ROWS * 2 * 4;
    static constexpr int BUDGET = 113 * 1024;     // two CTAs per SM
    static constexpr int STAGES_FIT = (BUDGET - MERGE_O_BYTES - MERGE_ML_BYTES - 128) / STAGE_BYTES;
    static constexpr int STAGES = STAGES_FIT > 5 ? 5 : STAGES_FIT;
    static_assert(STAGES >= kConsumerWarps, "every consumer warp needs a tile in flight");
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + MERGE_O_BYTES + MERGE_ML_BYTES + 128;
    static_assert(STAGES >= 2, "need at least a double buffer");
};

// D(16x8, f32) += A(16x16, f16, row) * B(16x8, f16, col)
__device__ __forceinline__ void mma_f16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// two E4M3 bytes (low byte first) -> two fp16 (exact)
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t two_bytes) {
    uint32_t r;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"((uint16_t)two_bytes));
    return r;
}
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
    __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// four bf16 (two 32-bit words) -> two fp16x2 words
__device__ __forceinline__ void bf16x4_to_f16x4(uint2 w, uint32_t& lo, uint32_t& hi) {
    lo = pack_f16x2(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xFFFF0000u));
    hi = pack_f16x2(__uint_as_float(w.y << 16), __uint_as_float(w.y & 0xFFFF0000u));
}

template <int ROWS>
__device__ __forceinline__ void decode_fp8_body(const CUtensorMap& tmK, const CUtensorMap& tmV,
                                                const DecodeFp8Params& pp, const DevSegment* segments,
                                                const int32_t* group_begin) {
    using C = Cfg8<ROWS>;
    constexpr int STAGES = C::STAGES;
    const DecodeParams& p = pp.base;

    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* stage_mem = smem;
    float* merge_o = reinterpret_cast<float*>(smem + STAGES * STAGE_BYTES);
    float* merge_ml = reinterpret_cast<float*>(smem + STAGES * STAGE_BYTES + C::MERGE_O_BYTES);
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES + C::MERGE_O_BYTES + C::MERGE_ML_BYTES);
    uint64_t* empty_bar = full_bar + STAGES;
    volatile int* give_up = reinterpret_cast<volatile int*>(empty_bar + STAGES);   // some thread ran out of patience
    static_assert(2 * STAGES * 8 + 4 <= 128, "barrier block");

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int seg_lo = group_begin[blockIdx.x], seg_hi = group_begin[blockIdx.x + 1];
    asm volatile("griddepcontrol.launch_dependents;");

    if ((smem_u32(smem) & 1023u) != 0) {   // the swizzle arithmetic below needs 1 KB alignment
        if (threadIdx.x == 0) atomicCAS(p.status, 0, status_word(kWaitMisaligned, linear_cta()));
        return;
    }
    const Abort ab{give_up, p.status, p.wait_limit_ns > 0 ? p.wait_limit_ns : kWaitLimitNs};
    if (threadIdx.x == 0) {
        *give_up = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);                 // released by the one warp that read the tile
        }
        mbar_fence_init();
    }
    __syncthreads();

    if (warp == kConsumerWarps) {
        // ------------------------------- producer ---------------------------------------
        if (lane == 0) {
            tma_prefetch_desc(&tmK);
            tma_prefetch_desc(&tmV);
            uint32_t it = 0;
            bool ok = true;
            for (int si = seg_lo; si < seg_hi && ok; ++si) {
                const DevSegment seg = segments[si];
                for (int k0 = seg.k_begin; k0 < seg.k_end; k0 += TILE_N, ++it) {
                    const uint32_t stage = it % STAGES, round = it / STAGES;
                    if (!wait_or_abort(&empty_bar[stage], (round & 1u) ^ 1u, ab, kWaitRingEmpty)) {
                        ok = false;
                        break;
                    }
                    uint8_t* kdst = stage_mem + stage * STAGE_BYTES;
                    mbar_expect_tx(&full_bar[stage], STAGE_BYTES);
                    const int row = seg.kv_row0 + (k0 - seg.k_begin);
                    tma_load_2d(kdst, &tmK, 0, row, &full_bar[stage]);
                    tma_load_2d(kdst + TENSOR_BYTES, &tmV, 0, row, &full_bar[stage]);
                }
            }
            // every copy this thread armed must have landed before it leaves (the CTA ends with its last
            // thread, and its shared memory then belongs to another CTA); at once when all went well
            const uint32_t in_flight = it < (uint32_t)STAGES ? it : (uint32_t)STAGES;
            for (uint32_t k = it - in_flight; k < it; ++k)
                if (!drain_wait(&full_bar[k % STAGES], (k / STAGES) & 1u, ab)) break;
        }
        return;
    }

    // ----------------------------------- consumers ---------------------------------------
    // Each consumer warp takes WHOLE tiles, round robin (tile number mod 4): per tile a warp then runs
    // one softmax for 64 keys instead of one per 16, which matters here because at half the bytes
    // per key the chain of dependent latencies per tile (products, shuffles, exponentials), not
    // the memory, would otherwise set the pace.  A tile is released by the one warp that read it.
    const int g = lane >> 2, tq = lane & 3;
    const int n_rows = p.rows_per_stream;
    // row address this lane supplies to ldmatrix.x4: matrix (lane >> 3) = (chunk pair member, key half)
    const int ld_key16 = ((lane >> 3) & 1) * 8 + (lane & 7);            // key row inside a 16-key group
    const int ld_chunk = lane >> 4;                                      // 0: first chunk of the pair, 1: second
    uint32_t it = 0;
    bool ok = true;

    for (int si = seg_lo; si < seg_hi; ++si) {
        const DevSegment seg = segments[si];
        const int head = seg.stream % pp.Hkv;
        const float sscale = pp.score_scale_log2[head], vscale = pp.v_scale[head];

        // Q as the fp16 A operand.  Reduction step ks covers channels 16 ks .. 16 ks + 15, and this
        // lane's four reduction slots (k = 2 tq, 2 tq + 1, 2 tq + 8, 2 tq + 9) stand for the four
        // consecutive channels 16 ks + 4 tq + {0, 1, 2, 3}: the order in which ldmatrix hands it K bytes.
        uint32_t qa[8][4];
        {
            const __nv_bfloat16* q0 = p.Q + ((int64_t)seg.q_row0 + g) * D + tq * 4;
            const __nv_bfloat16* q1 = q0 + 8 * D;
            const bool v0 = g < n_rows, v1 = ROWS == 16 && (g + 8) < n_rows;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const uint2 w0 = v0 ? *reinterpret_cast<const uint2*>(q0 + ks * 16) : make_uint2(0u, 0u);
                const uint2 w1 = v1 ? *reinterpret_cast<const uint2*>(q1 + ks * 16) : make_uint2(0u, 0u);
                bf16x4_to_f16x4(w0, qa[ks][0], qa[ks][2]);
                bf16x4_to_f16x4(w1, qa[ks][1], qa[ks][3]);
            }
        }
        const int n_full = seg.n_full;
        const int n_edge = min(n_full, seg.n_kv);      // tiles that end at or below it need no mask
        const int vis0 = min(seg.n_kv, max(0, n_full + (g % p.T)));
        const int vis1 = min(seg.n_kv, max(0, n_full + ((g + 8) % p.T)));

        float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
        float o[8][2][4];      // [16-channel chunk][even / odd channels][c fragment]
#pragma unroll
        for (int c = 0; c < 8; ++c)
#pragma unroll
            for (int h = 0; h < 2; ++h) o[c][h][0] = o[c][h][1] = o[c][h][2] = o[c][h][3] = 0.f;

        for (int k0 = seg.k_begin; k0 < seg.k_end; k0 += TILE_N, ++it) {
            if (!ok || (int)(it % kConsumerWarps) != warp) continue;       // not this warp's tile
            const uint32_t stage = it % STAGES, round = it / STAGES;
            if (!wait_or_abort(&full_bar[stage], round & 1u, ab, kWaitRingFull)) {
                ok = false;         // this warp touches no tile any more; it still walks to the barriers below
                continue;
            }
            const uint32_t kbase = smem_u32(stage_mem + stage * STAGE_BYTES);
            const uint32_t vbase = kbase + TENSOR_BYTES;

            // ---- S = Q K^T for 64 keys: four 16-key groups, two n-tiles of 8 keys each ----
            float s[8][4];
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
            for (int kg = 0; kg < 4; ++kg) {
                const int key = kg * 16 + ld_key16;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int chunk = 2 * j + ld_chunk;
                    uint32_t r0, r1, r2, r3;   // (keys 0-7, chunk 2j) (keys 8-15, 2j) (keys 0-7, 2j+1) (keys 8-15, 2j+1)
                    ldmatrix_x4(kbase + key * 128 + (((chunk ^ key) & 7) << 4), r0, r1, r2, r3);
                    mma_f16_16816(s[2 * kg], qa[2 * j], e4m3x2_to_f16x2(r0), e4m3x2_to_f16x2(r0 >> 16));
                    mma_f16_16816(s[2 * kg + 1], qa[2 * j], e4m3x2_to_f16x2(r1), e4m3x2_to_f16x2(r1 >> 16));
                    mma_f16_16816(s[2 * kg], qa[2 * j + 1], e4m3x2_to_f16x2(r2), e4m3x2_to_f16x2(r2 >> 16));
                    mma_f16_16816(s[2 * kg + 1], qa[2 * j + 1], e4m3x2_to_f16x2(r3), e4m3x2_to_f16x2(r3 >> 16));
                }
            }
            // ---- scale, mask (causal edge, sequence end, window start), online softmax ----
            const bool need_mask = k0 + TILE_N > n_edge || (p.window > 0 && k0 < n_full + p.T - 1 - p.window);
            int lo0 = -1, lo1 = -1;
            if (need_mask && p.window > 0) {
                lo0 = n_full + (g % p.T) - p.window;
                lo1 = n_full + ((g + 8) % p.T) - p.window;
            }
            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float v = s[nt][e] * sscale;
                    if (need_mask) {
                        const int j = k0 + nt * 8 + tq * 2 + (e & 1);
                        v = (j < ((e & 2) ? vis1 : vis0) && j >= ((e & 2) ? lo1 : lo0)) ? v : -INFINITY;
                    }
                    s[nt][e] = v;
                    if (e & 2) mx1 = fmaxf(mx1, v);
                    else mx0 = fmaxf(mx0, v);
                }
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
            const float mn0 = fmaxf(m0, mx0);
            const float ms0 = mn0 == -INFINITY ? 0.f : mn0;
            const float alpha0 = exp2f(m0 - ms0);
            m0 = mn0;
            float alpha1 = 1.f, ms1 = 0.f;
            if (ROWS == 16) {
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
                const float mn1 = fmaxf(m1, mx1);
                ms1 = mn1 == -INFINITY ? 0.f : mn1;
                alpha1 = exp2f(m1 - ms1);
                m1 = mn1;
            }
            // P in [0, 1], rounded to fp16, as the A operands of the four 16-key reduction steps
            uint32_t pa[4][4];
            float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
            for (int kg = 0; kg < 4; ++kg) {
                const float p00 = exp2f(s[2 * kg][0] - ms0), p01 = exp2f(s[2 * kg][1] - ms0);
                const float p10 = exp2f(s[2 * kg + 1][0] - ms0), p11 = exp2f(s[2 * kg + 1][1] - ms0);
                sum0 += (p00 + p01) + (p10 + p11);
                pa[kg][0] = pack_f16x2(p00, p01);
                pa[kg][2] = pack_f16x2(p10, p11);
                if (ROWS == 16) {
                    const float q00 = exp2f(s[2 * kg][2] - ms1), q01 = exp2f(s[2 * kg][3] - ms1);
                    const float q10 = exp2f(s[2 * kg + 1][2] - ms1), q11 = exp2f(s[2 * kg + 1][3] - ms1);
                    sum1 += (q00 + q01) + (q10 + q11);
                    pa[kg][1] = pack_f16x2(q00, q01);
                    pa[kg][3] = pack_f16x2(q10, q11);
                } else {
                    pa[kg][1] = pa[kg][3] = 0u;
                }
            }
            l0 = l0 * alpha0 + sum0;
            l1 = l1 * alpha1 + sum1;
            if (__any_sync(0xffffffffu, alpha0 != 1.f || alpha1 != 1.f)) {
#pragma unroll
                for (int c = 0; c < 8; ++c)
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        o[c][h][0] *= alpha0; o[c][h][1] *= alpha0;
                        o[c][h][2] *= alpha1; o[c][h][3] *= alpha1;
                    }
            }
            // ---- rows past the end of the sequence may hold anything (an FP8 NaN included):
            //      zero them so that 0 * garbage cannot produce NaN in O += P V ----
            if (k0 + TILE_N > seg.n_kv) {
                const int first_bad = max(seg.n_kv - k0, 0);          // 0..63
                uint8_t* vrow = stage_mem + stage * STAGE_BYTES + TENSOR_BYTES;
                if (lane < 8)
                    for (int r = first_bad; r < TILE_N; ++r)
                        *reinterpret_cast<uint4*>(vrow + r * 128 + lane * 16) = make_uint4(0u, 0u, 0u, 0u);
                __syncwarp();
            }
            // ---- O += P V.  The transposed ldmatrix hands this lane, for keys 2 tq and 2 tq + 1,
            //      the two channels 16 c + 2 g and 16 c + 2 g + 1: the even channels of a chunk
            //      form one n-tile, the odd ones the other ----
#pragma unroll
            for (int kg = 0; kg < 4; ++kg) {
                const int key = kg * 16 + ld_key16;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int chunk = 2 * j + ld_chunk;
                    uint32_t r0, r1, r2, r3;   // (keys 0-7, chunk 2j) (keys 8-15, 2j) (keys 0-7, 2j+1) (keys 8-15, 2j+1)
                    ldmatrix_x4_trans(vbase + key * 128 + (((chunk ^ key) & 7) << 4), r0, r1, r2, r3);
                    // bytes [k0 c0, k0 c1, k1 c0, k1 c1] -> [k0 c0, k1 c0 | k0 c1, k1 c1]
                    r0 = __byte_perm(r0, 0u, 0x3120);
                    r1 = __byte_perm(r1, 0u, 0x3120);
                    r2 = __byte_perm(r2, 0u, 0x3120);
                    r3 = __byte_perm(r3, 0u, 0x3120);
                    mma_f16_16816(o[2 * j][0], pa[kg], e4m3x2_to_f16x2(r0), e4m3x2_to_f16x2(r1));
                    mma_f16_16816(o[2 * j][1], pa[kg], e4m3x2_to_f16x2(r0 >> 16), e4m3x2_to_f16x2(r1 >> 16));
                    mma_f16_16816(o[2 * j + 1][0], pa[kg], e4m3x2_to_f16x2(r2), e4m3x2_to_f16x2(r3));
                    mma_f16_16816(o[2 * j + 1][1], pa[kg], e4m3x2_to_f16x2(r2 >> 16), e4m3x2_to_f16x2(r3 >> 16));
                }
            }
            if (k0 + TILE_N > seg.n_kv) fence_proxy_async_smem();   // generic writes before TMA reuse
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty_bar[stage]);
        }

        // ---- merge the four warps' states, write the final rows or this segment's partial ----
        l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
        l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
        if (ROWS == 16) {
            l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
            l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
        }
        {
            // accumulator (chunk c, even / odd tile, column 2 tq + j) is channel 16 c + 4 tq + 2 j (+ 1 if odd):
            // this lane's four values of a chunk are four consecutive channels
            float* mo = merge_o + (warp * ROWS) * D;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                *reinterpret_cast<float4*>(mo + g * D + c * 16 + tq * 4) =
                    make_float4(o[c][0][0], o[c][1][0], o[c][0][1], o[c][1][1]);
                if (ROWS == 16)
                    *reinterpret_cast<float4*>(mo + (g + 8) * D + c * 16 + tq * 4) =
                        make_float4(o[c][0][2], o[c][1][2], o[c][0][3], o[c][1][3]);
            }
            if (tq == 0) {
                merge_ml[(warp * ROWS + g) * 2] = m0;
                merge_ml[(warp * ROWS + g) * 2 + 1] = l0;
                if (ROWS == 16) {
                    merge_ml[(warp * ROWS + g + 8) * 2] = m1;
                    merge_ml[(warp * ROWS + g + 8) * 2 + 1] = l1;
                }
            }
        }
        named_barrier_sync(1, kConsumerWarps * 32);
        const bool final_out = seg.stream_nseg == 1 && !p.force_partial;
        for (int idx = threadIdx.x; idx < n_rows * D; idx += kConsumerWarps * 32) {
            const int r = idx / D, col = idx - r * D;
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < kConsumerWarps; ++w) M = fmaxf(M, merge_ml[(w * ROWS + r) * 2]);
            float L = 0.f, acc = 0.f;
            if (M != -INFINITY) {
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) {
                    const float f = exp2f(merge_ml[(w * ROWS + r) * 2] - M);
                    L += merge_ml[(w * ROWS + r) * 2 + 1] * f;
                    acc += merge_o[(w * ROWS + r) * D + col] * f;
                }
            }
            const float outv = L > 0.f ? acc / L * vscale : 0.f;
            const float lse = L > 0.f ? (M + log2f(L)) * 0.6931471805599453f : -INFINITY;
            if (final_out) {
                p.O[((int64_t)seg.q_row0 + r) * D + col] = __float2bfloat16(outv);
                if (p.lse && col == 0) p.lse[seg.q_row0 + r] = lse;
            } else {
                p.part_o[((int64_t)seg.slot * n_rows + r) * D + col] = outv;
                if (col == 0) p.part_lse[(int64_t)seg.slot * n_rows + r] = lse;
            }
        }
        named_barrier_sync(1, kConsumerWarps * 32);
    }
}

template <int ROWS>
__global__ void __launch_bounds__(kThreads, 2)
decode_fp8_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                  const __grid_constant__ DecodeFp8Params p) {
    decode_fp8_body<ROWS>(tmK, tmV, p, p.base.segments, p.base.group_begin);
}

// work tables as kernel parameters
template <int ROWS>
__global__ void __launch_bounds__(kThreads, 2)
decode_fp8_kernel_inline(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                         const __grid_constant__ DecodeFp8Params p, const __grid_constant__ DecodeInlineTables tab) {
    decode_fp8_body<ROWS>(tmK, tmV, p, tab.seg, tab.group_begin);
}

template <int ROWS>
cudaError_t launch_one(const DecodeFp8Params& p, const CUtensorMap& tmK, const CUtensorMap& tmV, int num_groups,
                       cudaStream_t stream, const DecodeInlineTables* tab) {
    if (tab)
        decode_fp8_kernel_inline<ROWS><<<num_groups, kThreads, Cfg8<ROWS>::SMEM_BYTES, stream>>>(tmK, tmV, p, *tab);
    else
        decode_fp8_kernel<ROWS><<<num_groups, kThreads, Cfg8<ROWS>::SMEM_BYTES, stream>>>(tmK, tmV, p);
    return cudaGetLastError();
}

template <int ROWS>
cudaError_t setup_one() {
    cudaError_t e = cudaFuncSetAttribute(decode_fp8_kernel<ROWS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         Cfg8<ROWS>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(decode_fp8_kernel_inline<ROWS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                Cfg8<ROWS>::SMEM_BYTES);
}

}  // namespace

cudaError_t decode_fp8_kernel_setup() {
    cudaError_t e = setup_one<8>();
    return e != cudaSuccess ? e : setup_one<16>();
}

cudaError_t launch_decode_fp8(const DecodeFp8Params& p, const CUtensorMap& tmK, const CUtensorMap& tmV,
                              int num_groups, cudaStream_t stream, const DecodeInlineTables* tab) {
    if (num_groups <= 0) return cudaSuccess;
    return p.base.rows_per_stream > 8 ? launch_one<16>(p, tmK, tmV, num_groups, stream, tab)
                                      : launch_one<8>(p, tmK, tmV, num_groups, stream, tab);
}

}  // namespace yoco
