// Writing the shared cache: K^ = RMSNorm(X) W_K, V^ = RMSNorm(X) W_V for the T new tokens of every
// sequence, stored straight into the head-major cache rows [N_i - T, N_i) that the cross-decoder
// attention reads.
//
// RMSNorm(x) = x * r * g with r = 1 / sqrt(mean(x^2) + eps).  The gain g is folded into the weights
// once (fold_gain_kernel: Wg = g (.) W, weights do not change between calls) and r is a per-row
// scalar, so the product is a plain GEMM X Wg whose rows are scaled by r at the end:
//   one CTA = 128 tokens x 128 output channels (one KV head of K^ or of V^ when d = 128), K loop
//   over d_model in steps of 128 through a three-stage TMA ring, tcgen05.mma with the accumulator
//   in tensor memory.  While a stage of X sits in shared memory the epilogue warps add up the
//   squares of their rows from it, so X is read once and there is no separate normalisation pass.
// Roles (192 threads): warp 0 TMA producer, warp 1 MMA issuer (whole warp walks, one elected lane
// issues), warps 2-5 row statistics during the loop, then scale / round to bf16 / scatter.
// Every wait is bounded and reports through the status word.
#include <cuda_fp8.h>

#include <algorithm>

#include "kernels.h"
#include "ptx.cuh"
#include "tcgen05.cuh"

namespace yoco {

// Status word of the append kernel (it takes no workspace): 0, or the code of a bounded wait that
// ran out.  Sticky until read_and_clear_kv_append_status().
__device__ int32_t g_kv_append_status;

namespace {

constexpr int BM = 128, BN = 128, BK = 128;
constexpr int kThreads = 192;
constexpr int HALF_BYTES = 128 * 128;            // 128 rows x 64 bf16: one swizzled half tile
constexpr int TILE_BYTES = 2 * HALF_BYTES;       // an X tile [128 tokens, 128 k] or a W tile [128 k, 128 n]
constexpr int STAGES = 3;
constexpr int STAGE_BYTES = 2 * TILE_BYTES;
constexpr int OFF_BAR = STAGES * STAGE_BYTES;
constexpr int SMEM_BYTES = OFF_BAR + (2 * STAGES + 2) * 8 + 16;
constexpr uint32_t TMEM_COLS = 128;

// FP8 = false: rows stored as bf16.  FP8 = true: rows divided by the head's scale and stored as FP8
// E4M3 bytes (round to nearest even, saturating at +-448), one byte per element.
template <bool FP8>
__global__ void __launch_bounds__(kThreads, 1)
kv_append_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmWk,
                 const __grid_constant__ CUtensorMap tmWv, const KvAppendParams p,
                 const __grid_constant__ KvAppendTables tab, const __grid_constant__ KvAppendScales sc) {
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + OFF_BAR);   // [STAGES] tile pair has landed
    uint64_t* empty = full + STAGES;                                // [STAGES] MMA and row sums are done with it
    uint64_t* acc_full = empty + STAGES;                            // accumulator complete
    uint64_t* drain_bar = acc_full + 1;                             // everything the issuer started has finished
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain_bar + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * BN;          // first output column (K^ columns, then V^ columns)
    const int m0 = blockIdx.y * BM;          // first token
    const int KT = p.d_model / BK;
    const Abort ab{abort_flag, &g_kv_append_status, kWaitLimitNs};
    const bool aligned_ok = (smem_u32(smem) & 1023u) == 0;

    if (threadIdx.x == 0) {
        *abort_flag = aligned_ok ? 0 : 1;
        if (!aligned_ok) atomicCAS(&g_kv_append_status, 0, status_word(kWaitMisaligned, linear_cta()));
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1 + 4);     // one tcgen05.commit + four row-sum warps
        }
        mbar_init(acc_full, 1);
        mbar_init(drain_bar, 1);
        mbar_fence_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_acc = *tmem_slot;

    if (warp == 0) {
        // ======================================= TMA producer ================================
        if (lane == 0 && aligned_ok) {
            const bool is_v = n0 >= p.n_half;
            const CUtensorMap* tmW = is_v ? &tmWv : &tmWk;
            const int nw = n0 - (is_v ? p.n_half : 0);
            tma_prefetch_desc(&tmX);
            tma_prefetch_desc(tmW);
            int armed = 0;                                   // copies started, for the drain on the way out
            for (int kt = 0; kt < KT; ++kt, ++armed) {
                const uint32_t s = kt % STAGES, ph = (kt / STAGES) & 1u;
                if (!wait_or_abort(&empty[s], ph ^ 1u, ab, kWaitRingEmpty)) break;
                uint8_t* a = smem + s * STAGE_BYTES;
                uint8_t* b = a + TILE_BYTES;
                mbar_expect_tx(&full[s], STAGE_BYTES);
                for (int h = 0; h < 2; ++h) {
                    tma_load_2d(a + h * HALF_BYTES, &tmX, kt * BK + h * 64, m0, &full[s]);
                    tma_load_2d(b + h * HALF_BYTES, tmW, nw + h * 64, kt * BK, &full[s]);
                }
            }
            // every copy this thread started must have landed before the CTA may end
            for (int k = armed > STAGES ? armed - STAGES : 0; k < armed; ++k)
                if (!drain_wait(&full[k % STAGES], (uint32_t)(k / STAGES) & 1u, ab)) break;
        }
    } else if (warp == 1) {
        // ======================================= MMA issuer ==================================
        if (aligned_ok) {
            constexpr uint32_t idesc = make_idesc(BN, true);
            const uint32_t sbase = smem_u32(smem);
            bool ok = true;
            for (int kt = 0; kt < KT && ok; ++kt) {
                const uint32_t s = kt % STAGES, ph = (kt / STAGES) & 1u;
                if (!(ok = warp_wait(&full[s], ph, ab, kWaitRingFull))) break;
                tc_fence_after();
                const uint32_t a_lo = desc_lo(sbase + s * STAGE_BYTES, 16);
                const uint32_t b_lo = desc_lo(sbase + s * STAGE_BYTES + TILE_BYTES, BK * 128);
                if (elect_one()) {
#pragma unroll
                    for (int ks = 0; ks < BK / 16; ++ks) {
                        const uint32_t a_off = ((ks >> 2) * HALF_BYTES + (ks & 3) * 32) >> 4;
                        const uint32_t b_off = (uint32_t)(ks * 16 * 128) >> 4;
                        umma_ss(tmem_acc, desc_from_lo(a_lo + a_off, 1024), desc_from_lo(b_lo + b_off, 1024), idesc,
                                (kt > 0 || ks > 0) ? 1u : 0u);
                    }
                    umma_commit(&empty[s]);
                    if (kt == KT - 1) umma_commit(acc_full);
                }
                __syncwarp();
            }
            // nothing this warp issued may still be running when tensor memory is released and the CTA ends
            if (elect_one()) {
                umma_commit(drain_bar);
                drain_wait(drain_bar, 0u, ab);
            }
            __syncwarp();
        }
    } else {
        // ============================ row statistics, then epilogue ==========================
        const int quad = warp & 3;                     // TMEM lane quadrant this warp may access
        const int row = quad * 32 + lane;              // token row inside the tile
        const int m = m0 + row;
        bool ok = aligned_ok;
        float ss = 0.f;                                // sum of squares of this token's hidden state
        for (int kt = 0; kt < KT; ++kt) {
            if (!ok) continue;
            const uint32_t s = kt % STAGES, ph = (kt / STAGES) & 1u;
            if (!(ok = warp_wait(&full[s], ph, ab, kWaitRingFull))) continue;
            const uint8_t* a = smem + s * STAGE_BYTES + row * 128;
            float part[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    // the swizzle only permutes the 16-byte chunks of a row: any order will do, and
                    // starting each thread at a different chunk spreads the banks
                    const uint4 v = *reinterpret_cast<const uint4*>(a + h * HALF_BYTES + (((c + row) & 7) << 4));
                    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float lo = __uint_as_float(w[q] << 16), hi = __uint_as_float(w[q] & 0xFFFF0000u);
                        part[q] = fmaf(lo, lo, part[q]);
                        part[q] = fmaf(hi, hi, part[q]);
                    }
                }
            ss += (part[0] + part[1]) + (part[2] + part[3]);
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);
        }
        if (ok) ok = warp_wait(acc_full, 0u, ab, kWaitTensor);
        if (ok) {
            tc_fence_after();
            const float r = 1.f / sqrtf(ss / (float)p.d_model + p.eps);
            const int i = m / p.T, t = m - i * p.T;
            const bool valid = m < p.M;
            const int64_t row0 = valid ? (int64_t)tab.row0[i] + t : 0;
            const int head_rows = valid ? tab.head_rows[i] : 0;
#pragma unroll
            for (int cb = 0; cb < BN / 32; ++cb) {
                float o[32];
                tmem_ld32(tmem_acc + ((uint32_t)(quad * 32) << 16) + cb * 32, o);
                tmem_wait_ld();
                if (valid) {
                    const int n = n0 + cb * 32;
                    const bool is_v = n >= p.n_half;
                    const int nn = n - (is_v ? p.n_half : 0);
                    const int c = nn / p.d, e = nn - c * p.d;
                    if (FP8) {
                        const float rs = r * (is_v ? sc.inv_v[c] : sc.inv_k[c]);
                        uint8_t* dst8 = reinterpret_cast<uint8_t*>(is_v ? p.V : p.K) + (row0 + (int64_t)c * head_rows) * p.d + e;
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            uint32_t w[4];
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const uint32_t lo = __nv_cvt_float2_to_fp8x2(
                                    make_float2(o[q * 16 + k * 4 + 0] * rs, o[q * 16 + k * 4 + 1] * rs), __NV_SATFINITE, __NV_E4M3);
                                const uint32_t hi = __nv_cvt_float2_to_fp8x2(
                                    make_float2(o[q * 16 + k * 4 + 2] * rs, o[q * 16 + k * 4 + 3] * rs), __NV_SATFINITE, __NV_E4M3);
                                w[k] = lo | (hi << 16);
                            }
                            *reinterpret_cast<uint4*>(dst8 + q * 16) = make_uint4(w[0], w[1], w[2], w[3]);
                        }
                        continue;
                    }
                    __nv_bfloat16* dst = (is_v ? p.V : p.K) + (row0 + (int64_t)c * head_rows) * p.d + e;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint4 pk;
                        pk.x = pack_bf16x2(o[q * 8 + 0] * r, o[q * 8 + 1] * r);
                        pk.y = pack_bf16x2(o[q * 8 + 2] * r, o[q * 8 + 3] * r);
                        pk.z = pack_bf16x2(o[q * 8 + 4] * r, o[q * 8 + 5] * r);
                        pk.w = pack_bf16x2(o[q * 8 + 6] * r, o[q * 8 + 7] * r);
                        *reinterpret_cast<uint4*>(dst + q * 8) = pk;
                    }
                }
            }
            tc_fence_before();
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_acc, TMEM_COLS);
    }
}

// ---- a decode step: at most 16 tokens ---------------------------------------------------------
// With a handful of rows the product is a stream of the two weight matrices (33 MB at d_model 4,096
// and 2 x 1,024 output channels) and the 128-row tensor-core tile above would leave all but
// Hkv * d / 64 SMs idle.  Here a CTA owns 64 output channels and 1/S of d_model; the S CTAs of a
// cluster cover d_model between them, each with its whole weight slab in flight at once (up to four
// 16 KB TMA boxes), multiply with mma.sync (the tokens are the 16 rows of the A operand, the slab goes
// through ldmatrix.trans), and add their partial sums and their partial row sums of squares through
// distributed shared memory: CTA j of the cluster reduces and stores 64 / S of the channels.
constexpr int SK_THREADS = 128;
constexpr int SK_COLS = 64;                      // output channels per CTA: one TMA box wide
constexpr int SK_KBOX = 128;                     // weight rows per TMA box
constexpr int SK_STAGES = 4;
constexpr int SK_ROWS = 16;
constexpr int SK_XSTRIDE = SK_KBOX + 8;          // bf16 elements per X row in shared memory (conflict-free)
constexpr int SK_OFF_X = SK_STAGES * HALF_BYTES;
constexpr int SK_OFF_RED = SK_OFF_X + SK_ROWS * SK_XSTRIDE * 2;
constexpr int SK_OFF_SSQ = SK_OFF_RED + SK_ROWS * SK_COLS * 4;
constexpr int SK_OFF_BAR = SK_OFF_SSQ + SK_ROWS * 4;
constexpr int SK_SMEM_BYTES = SK_OFF_BAR + SK_STAGES * 8 + 16;

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ float ld_cluster_f(uint32_t addr) {
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}

// grid = (Hkv*d / 64, 2 (K^ | V^), S), cluster (1, 1, S); S * n_chunks * 128 = d_model
template <bool FP8>
__global__ void __launch_bounds__(SK_THREADS)
kv_append_small_kernel(const __grid_constant__ CUtensorMap tmWk, const __grid_constant__ CUtensorMap tmWv,
                       const KvAppendParams p, const __grid_constant__ KvAppendTables tab,
                       const __grid_constant__ KvAppendScales sc) {
    extern __shared__ __align__(1024) uint8_t smem[];
    __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(smem + SK_OFF_X);
    float* red = reinterpret_cast<float*>(smem + SK_OFF_RED);      // [16][64] partial sums of this CTA
    float* ssq = reinterpret_cast<float*>(smem + SK_OFF_SSQ);      // [16] partial sums of squares
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + SK_OFF_BAR);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;
    const int S = (int)gridDim.z;
    const int rank = (int)cluster_ctarank();
    const bool is_v = blockIdx.y != 0;
    const int col0 = blockIdx.x * SK_COLS;                 // first channel inside K^ (or V^)
    const int k_slice = p.d_model / S;
    const int k_base = rank * k_slice;
    const int n_chunks = k_slice / SK_KBOX;
    const CUtensorMap* tmW = is_v ? &tmWv : &tmWk;
    bool ok = (smem_u32(smem) & 1023u) == 0;
    if (!ok && threadIdx.x == 0) atomicCAS(&g_kv_append_status, 0, status_word(kWaitMisaligned, linear_cta()));
    volatile int* give_up = reinterpret_cast<volatile int*>(full + SK_STAGES);   // behind the barriers
    const Abort ab{give_up, &g_kv_append_status, kWaitLimitNs};
    int armed = 0;                                          // thread 0: copies started

    if (threadIdx.x == 0) {
        *give_up = 0;
        for (int s = 0; s < SK_STAGES; ++s) mbar_init(&full[s], 1);
        mbar_fence_init();
    }
    __syncthreads();
    if (threadIdx.x == 0 && ok) {
        tma_prefetch_desc(tmW);
        for (int c = 0; c < n_chunks && c < SK_STAGES; ++c, ++armed) {
            mbar_expect_tx(&full[c], HALF_BYTES);
            tma_load_2d(smem + c * HALF_BYTES, tmW, col0, k_base + c * SK_KBOX, &full[c]);
        }
    }

    float acc[2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
    float sq = 0.f;                                         // this thread's share of a row's sum of squares
    const int xr = threadIdx.x >> 3, xc = (threadIdx.x & 7) * 16;   // X staging: row, first of 16 elements

    // this thread's 16 elements of X[:, chunk]; the next chunk's are requested one iteration ahead, so
    // that only the first load's latency is exposed
    const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
    const uint4* xsrc = reinterpret_cast<const uint4*>(p.X + (int64_t)(xr < p.M ? xr : 0) * p.d_model + k_base + xc);
    uint4 v0 = zero4, v1 = zero4;
    if (xr < p.M && n_chunks > 0) {
        v0 = xsrc[0];
        v1 = xsrc[1];
    }
    for (int c = 0; c < n_chunks; ++c) {
        // X[:, chunk] -> shared memory (rows beyond M are zero), squares on the way
        uint4 nv0 = zero4, nv1 = zero4;
        if (xr < p.M && c + 1 < n_chunks) {
            nv0 = xsrc[(c + 1) * (SK_KBOX / 8)];
            nv1 = xsrc[(c + 1) * (SK_KBOX / 8) + 1];
        }
        {
            const uint32_t w[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float a = __uint_as_float(w[j] << 16), b = __uint_as_float(w[j] & 0xFFFF0000u);
                sq = fmaf(a, a, sq);
                sq = fmaf(b, b, sq);
            }
            uint4* dst = reinterpret_cast<uint4*>(xs + xr * SK_XSTRIDE + xc);
            dst[0] = v0;
            dst[1] = v1;
        }
        __syncthreads();
        const int stage = c % SK_STAGES;
        if (ok && !wait_or_abort(&full[stage], (uint32_t)(c / SK_STAGES) & 1u, ab, kWaitRingFull)) ok = false;
        if (ok) {
            const uint32_t wbase = smem_u32(smem + stage * HALF_BYTES);
            const int k_l = ((lane >> 3) & 1) * 8 + (lane & 7);      // ldmatrix row inside a 16-k step
            const int chunk16 = warp * 2 + (lane >> 4);              // 16-byte column chunk: 8 channels
#pragma unroll
            for (int ks = 0; ks < SK_KBOX / 16; ++ks) {
                uint32_t a[4];
                const __nv_bfloat16* x0 = xs + g * SK_XSTRIDE + ks * 16 + tq * 2;
                a[0] = *reinterpret_cast<const uint32_t*>(x0);
                a[1] = *reinterpret_cast<const uint32_t*>(x0 + 8 * SK_XSTRIDE);
                a[2] = *reinterpret_cast<const uint32_t*>(x0 + 8);
                a[3] = *reinterpret_cast<const uint32_t*>(x0 + 8 * SK_XSTRIDE + 8);
                const int krow = ks * 16 + k_l;
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4_trans(wbase + krow * 128 + (((chunk16 ^ krow) & 7) << 4), b0, b1, b2, b3);
                mma_bf16_16816(acc[0], a, b0, b1);
                mma_bf16_16816(acc[1], a, b2, b3);
            }
        }
        __syncthreads();                                    // everyone is done with xs and with the stage
        if (threadIdx.x == 0 && ok && c + SK_STAGES < n_chunks) {
            fence_proxy_async_smem();
            mbar_expect_tx(&full[stage], HALF_BYTES);
            tma_load_2d(smem + stage * HALF_BYTES, tmW, col0, k_base + (c + SK_STAGES) * SK_KBOX, &full[stage]);
            ++armed;
        }
        v0 = nv0;
        v1 = nv1;
    }

    // partial results of this CTA -> its shared memory
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
        const int col = warp * 16 + nt * 8 + tq * 2;
        *reinterpret_cast<float2*>(red + g * SK_COLS + col) = make_float2(acc[nt][0], acc[nt][1]);
        *reinterpret_cast<float2*>(red + (g + 8) * SK_COLS + col) = make_float2(acc[nt][2], acc[nt][3]);
    }
    sq += __shfl_xor_sync(0xffffffffu, sq, 1);
    sq += __shfl_xor_sync(0xffffffffu, sq, 2);
    sq += __shfl_xor_sync(0xffffffffu, sq, 4);
    if ((threadIdx.x & 7) == 0) ssq[xr] = sq;
    cluster_sync_all();

    // CTA `rank` adds up and stores channels [rank * cw, (rank + 1) * cw) of the 64, eight per thread
    const int cw = SK_COLS / S;                             // 8, 16, 32 or 64
    const int groups = cw / 8;
    if (threadIdx.x < SK_ROWS * groups) {
        const int row = threadIdx.x / groups, cg = threadIdx.x - row * groups;
        const int col = rank * cw + cg * 8;
        if (row < p.M) {
            float v[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            float total_sq = 0.f;
            const uint32_t red_addr = smem_u32(red + row * SK_COLS + col);
            const uint32_t ssq_addr = smem_u32(ssq + row);
            // all remote loads first, then the sums: a load-add-load chain would pay S round trips
            float4 lo[8], hi[8];
            float part_sq[8];
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                if (r < S) {
                    lo[r] = ld_cluster_f4(map_to_rank(red_addr, r));
                    hi[r] = ld_cluster_f4(map_to_rank(red_addr + 16, r));
                    part_sq[r] = ld_cluster_f(map_to_rank(ssq_addr, r));
                }
            }
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                if (r < S) {
                    v[0] += lo[r].x; v[1] += lo[r].y; v[2] += lo[r].z; v[3] += lo[r].w;
                    v[4] += hi[r].x; v[5] += hi[r].y; v[6] += hi[r].z; v[7] += hi[r].w;
                    total_sq += part_sq[r];
                }
            }
            const float rn = rsqrtf(total_sq / (float)p.d_model + p.eps);
            const int i = row / p.T, t = row - i * p.T;
            const int n = col0 + col;                       // channel inside K^ (or V^)
            const int head = n / p.d, e = n - head * p.d;
            const int64_t dst_row = (int64_t)tab.row0[i] + t + (int64_t)head * tab.head_rows[i];
            if (FP8) {
                const float rs = rn * (is_v ? sc.inv_v[head] : sc.inv_k[head]);
                uint32_t w[2];
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const uint32_t lo16 = __nv_cvt_float2_to_fp8x2(make_float2(v[4 * j] * rs, v[4 * j + 1] * rs), __NV_SATFINITE, __NV_E4M3);
                    const uint32_t hi16 = __nv_cvt_float2_to_fp8x2(make_float2(v[4 * j + 2] * rs, v[4 * j + 3] * rs), __NV_SATFINITE, __NV_E4M3);
                    w[j] = lo16 | (hi16 << 16);
                }
                uint8_t* dst8 = reinterpret_cast<uint8_t*>(is_v ? p.V : p.K) + dst_row * p.d + e;
                *reinterpret_cast<uint2*>(dst8) = make_uint2(w[0], w[1]);
            } else {
                uint4 pk;
                pk.x = pack_bf16x2(v[0] * rn, v[1] * rn);
                pk.y = pack_bf16x2(v[2] * rn, v[3] * rn);
                pk.z = pack_bf16x2(v[4] * rn, v[5] * rn);
                pk.w = pack_bf16x2(v[6] * rn, v[7] * rn);
                *reinterpret_cast<uint4*>((is_v ? p.V : p.K) + dst_row * p.d + e) = pk;
            }
        }
    }
    // every copy thread 0 started must have landed before the CTA may end (at once unless a wait gave up)
    if (threadIdx.x == 0)
        for (int k = armed > SK_STAGES ? armed - SK_STAGES : 0; k < armed; ++k)
            if (!drain_wait(&full[k % SK_STAGES], (uint32_t)(k / SK_STAGES) & 1u, ab)) break;
    cluster_sync_all();                                     // nobody leaves while its memory is being read
}

// Wg[k, n] = g[k] * W[k, n]: the product of two bf16 values is exact in fp32, one rounding to bf16.
__global__ void fold_gain_kernel(const __nv_bfloat16* __restrict__ g, const __nv_bfloat16* __restrict__ W,
                                 __nv_bfloat16* __restrict__ Wg, int64_t d_model, int64_t n_out) {
    const int64_t total = d_model * n_out;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t k = idx / n_out;
        Wg[idx] = __float2bfloat16(__bfloat162float(g[k]) * __bfloat162float(W[idx]));
    }
}

}  // namespace

cudaError_t read_and_clear_kv_append_status(int32_t* word, cudaStream_t stream) {
    cudaError_t e = cudaMemcpyFromSymbolAsync(word, g_kv_append_status, sizeof(int32_t), 0, cudaMemcpyDeviceToHost, stream);
    if (e != cudaSuccess) return e;
    if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return e;
    if (*word == 0) return cudaSuccess;
    const int32_t zero = 0;
    e = cudaMemcpyToSymbolAsync(g_kv_append_status, &zero, sizeof zero, 0, cudaMemcpyHostToDevice, stream);
    return e != cudaSuccess ? e : cudaStreamSynchronize(stream);
}

cudaError_t kv_append_kernel_setup() {
    cudaError_t e = cudaFuncSetAttribute(kv_append_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(kv_append_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES)) != cudaSuccess)
        return e;
    if ((e = cudaFuncSetAttribute(kv_append_small_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  SK_SMEM_BYTES)) != cudaSuccess)
        return e;
    return cudaFuncSetAttribute(kv_append_small_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SK_SMEM_BYTES);
}

cudaError_t launch_kv_append(const KvAppendParams& p, const KvAppendTables& tab, const CUtensorMap& tmX,
                             const CUtensorMap& tmWk, const CUtensorMap& tmWv, cudaStream_t stream,
                             const KvAppendScales* fp8_scales) {
    if (p.M <= 0) return cudaSuccess;
    if (p.M <= SK_ROWS && p.n_half % SK_COLS == 0 && p.d_model % SK_KBOX == 0) {
        // a decode step: stream the weights with clusters that split d_model
        int S = 8;
        while (S > 1 && p.d_model % (S * SK_KBOX) != 0) S /= 2;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(p.n_half / SK_COLS), 2u, (unsigned)S);
        cfg.blockDim = dim3(SK_THREADS);
        cfg.dynamicSmemBytes = SK_SMEM_BYTES;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 1;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = (unsigned)S;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        KvAppendScales none{};
        if (fp8_scales) return cudaLaunchKernelEx(&cfg, kv_append_small_kernel<true>, tmWk, tmWv, p, tab, *fp8_scales);
        return cudaLaunchKernelEx(&cfg, kv_append_small_kernel<false>, tmWk, tmWv, p, tab, none);
    }
    dim3 grid((unsigned)(2 * p.n_half / BN), (unsigned)((p.M + BM - 1) / BM));
    if (fp8_scales) {
        kv_append_kernel<true><<<grid, kThreads, SMEM_BYTES, stream>>>(tmX, tmWk, tmWv, p, tab, *fp8_scales);
    } else {
        KvAppendScales none{};
        kv_append_kernel<false><<<grid, kThreads, SMEM_BYTES, stream>>>(tmX, tmWk, tmWv, p, tab, none);
    }
    return cudaGetLastError();
}

cudaError_t launch_fold_gain(const __nv_bfloat16* g, const __nv_bfloat16* W, __nv_bfloat16* Wg, int64_t d_model,
                             int64_t n_out, cudaStream_t stream) {
    const int64_t total = d_model * n_out;
    if (total <= 0) return cudaSuccess;
    const int blocks = (int)std::min<int64_t>((total + 255) / 256, 148 * 8);
    fold_gain_kernel<<<blocks, 256, 0, stream>>>(g, W, Wg, d_model, n_out);
    return cudaGetLastError();
}

}  // namespace yoco
