// Multi-token chunk / full-sequence attention on the tcgen05 tensor cores, two row tiles per CTA.
//
// One CTA owns 256 of the G*T query rows of a (sequence, KV head) stream, as two 128-row tiles
// that share every K/V tile brought into shared memory, and walks a contiguous range of 128-key
// tiles.  Three warpgroups (384 threads):
//   warpgroup 0   warp 0 = TMA producer (both Q tiles once per segment; K through a three-deep and
//                 V through a two-deep ring), warps 1 and 2 = issuers of all tensor-core products of
//                 row tiles 0 and 1; gives most of its registers away
//   warpgroup 1   softmax of row tile 0 (thread = query row)
//   warpgroup 2   softmax of row tile 1
// Every 128-key tile is processed as two 64-key half steps.  Tensor memory (512 columns):
//   S_0^0 S_0^1 | S_1^0 S_1^1 | O_0 | O_1      (64 fp32 columns per S buffer, 128 per O)
// S_r^h receives the scores of row tile r against half h of the key tile, so the scores of the
// next half step are already being computed while a warpgroup works on the current one.  A softmax
// thread reads its S row, keeps the running max / sum, and writes P (bf16, two per 32-bit column)
// over the first 32 columns of the same S buffer; O_r += P_r V then takes P straight from tensor
// memory as the A operand, so P never touches shared memory.  The issuer of a row tile puts the
// next score product of a buffer right behind the P V product that reads it: the tensor pipe runs
// the products of one thread in the order issued, so the buffer needs no barrier round trip between
// the two.  O in tensor memory is rescaled only when a row max outgrew the reference by more than 2^8.
// Every wait is bounded and reports through the status word.
//
// FP8 = true reads an 8-bit cache (FP8 E4M3 bytes, one fp32 scale per KV head, head dimension 128):
// the producer brings a 128-key tile of bytes (16 KB) into the upper half of a ring stage, a fourth
// warpgroup (512 threads then; one warp per scheduler, 32 rows of every tile each)
// widens it in place to fp16 in the layout the tensor-core descriptors read (every E4M3 value is an
// fp16 value, so this is exact; row r of the bytes sits exactly where row r of the second 64-channel
// half goes, so a thread only ever overwrites its own source row), Q is converted bf16 -> fp16 in
// place once per segment, P is rounded to fp16, and all products run fp16 x fp16.  k_scale folds
// into the softmax scale, v_scale multiplies the normalised output.
#include <cuda_fp16.h>

#include "kernels.h"
#include "ptx.cuh"
#include "tcgen05.cuh"

namespace yoco {

namespace {

constexpr int BM = 128;                        // rows of one tensor-core tile
constexpr int BN = kChunkTileN;                // 128 keys per shared-memory tile
constexpr int BH = BN / 2;                     // keys per half step
// three warpgroups for a bf16 cache; a fourth one widens the tiles of an 8-bit cache
template <bool FP8>
constexpr int kThreadsOf = FP8 ? 512 : 384;
constexpr int HALF_BYTES = 128 * 128;          // 128 rows x 64 bf16: one swizzled half tile
constexpr uint32_t TMEM_COLS = 512;
constexpr float kRescaleThreshold = 8.f;       // in log2 units: P stays below 2^8
// Register split after launch.  The CTA starts with what its thread count allows (168 registers per
// thread for 384 threads, 128 for 512); warpgroup 0 (and the widening warpgroup) give back down to
// kOther / kWiden and the softmax warpgroups grow to kSoftmax.  The total must fit in what the CTA
// was launched with, or the request to grow would never be granted.
template <bool FP8>
struct Regs {
    static constexpr int kLaunch = FP8 ? 128 : 168, kSoftmax = FP8 ? 192 : 224, kOther = 56, kWiden = 64;
    static_assert(128 * kOther + 256 * kSoftmax + (FP8 ? 128 * kWiden : 0) <= kLaunch * kThreadsOf<FP8>,
                  "register pool of the CTA");
};

template <int D>
struct PCfg {
    static constexpr int HALVES = D / 64;
    static constexpr int TILE_BYTES = HALVES * HALF_BYTES;     // one Q, K or V tile
    static constexpr int K_STAGES = 3, V_STAGES = 2;
    static constexpr int OFF_Q = 0;                            // two tiles
    static constexpr int OFF_K = OFF_Q + 2 * TILE_BYTES;
    static constexpr int OFF_V = OFF_K + K_STAGES * TILE_BYTES;
    static constexpr int OFF_BAR = OFF_V + V_STAGES * TILE_BYTES;
    static constexpr int NUM_BARS = 2 + 2 * K_STAGES + 2 * V_STAGES + 12 + 3 + (K_STAGES + V_STAGES + 1);
    static constexpr int SMEM_BYTES = OFF_BAR + NUM_BARS * 8 + 16;
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory");
};

// Which of the 16 score pairs of a 32-key chunk take their exponential on the FMA pipe (a cubic, see
// f2_exp2_poly) instead of the special-function unit (16 results per clock per SM), spread evenly so
// that the two instruction streams interleave.  Measured on the 32K-cache chunk case with the turns
// described below in place, 0 / 2 / 4 of 16: 974 / 1,055 / 1,125 TFLOP/s.
constexpr int kPolyPairs = 4;
__host__ __device__ constexpr bool poly_pair(int j) {
    return ((j + 1) * kPolyPairs) / 16 != (j * kPolyPairs) / 16;
}

__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
    __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// two E4M3 bytes (low byte first) -> two fp16 (exact)
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t two_bytes) {
    uint32_t r;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"((uint16_t)two_bytes));
    return r;
}
// two bf16 -> two fp16 (round to nearest; |x| < 65504 required of Q)
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t w) {
    return pack_f16x2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
}

template <int D, bool FP8>
__global__ void __launch_bounds__(kThreadsOf<FP8>, 1)
chunk_pair_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV, const ChunkParams p,
                  const __grid_constant__ ChunkFp8Scales sc) {
    static_assert(!FP8 || D == 128, "the 8-bit cache path is built for head dimension 128");
    using C = PCfg<D>;
    constexpr int HALVES = C::HALVES;
    constexpr int KS = C::K_STAGES, VS = C::V_STAGES;
    constexpr int KSTEPS_QK = D / 16;
    constexpr int KSTEPS_PV = BH / 16;

    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BAR);
    uint64_t* q_full = bars + 0;
    uint64_t* q_empty = bars + 1;
    uint64_t* k_full = bars + 2;             // [KS]
    uint64_t* k_empty = k_full + KS;         // [KS]
    uint64_t* v_full = k_empty + KS;         // [VS]
    uint64_t* v_empty = v_full + VS;         // [VS]
    uint64_t* s_full = v_empty + VS;         // [2][2]  S_r^h holds the scores of the current half step
    uint64_t* p_full = s_full + 4;           // [2][2]  P_r^h has been written over S_r^h
    uint64_t* pv_done = p_full + 4;          // [2][2]  O_r includes the current half step; P_r^h is dead
    uint64_t* drain_bar = pv_done + 4;       // [3]     everything issuer warp 1 + i started has finished
    uint64_t* k_ready = drain_bar + 3;       // [KS]    8-bit cache: the K tile has been widened to fp16
    uint64_t* v_ready = k_ready + KS;        // [VS]    ... the V tile
    uint64_t* q_ready = v_ready + VS;        //         ... both Q tiles have been converted to fp16
    // what the issuers and the softmax warpgroups wait on for an operand tile
    uint64_t* k_use = FP8 ? k_ready : k_full;
    uint64_t* v_use = FP8 ? v_ready : v_full;
    uint64_t* q_use = FP8 ? q_ready : q_full;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + C::NUM_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int group = blockIdx.x / p.m_tiles, m_tile = blockIdx.x - group * p.m_tiles;
    const int seg_lo = p.group_begin[group], seg_hi = p.group_begin[group + 1];
    const Abort ab{abort_flag, p.status, kWaitLimitNs};
    const bool aligned_ok = (smem_u32(smem) & 1023u) == 0;

    if (threadIdx.x == 0) {
        *abort_flag = aligned_ok ? 0 : 1;
        if (!aligned_ok) atomicCAS(p.status, 0, status_word(kWaitMisaligned, linear_cta()));
        mbar_init(q_full, 1);
        mbar_init(q_empty, 2);
        for (int b = 0; b < 3; ++b) mbar_init(&drain_bar[b], 1);
        for (int b = 0; b < KS + VS + 1; ++b) mbar_init(&k_ready[b], 4);      // the four widening warps
        for (int b = 0; b < KS; ++b) {
            mbar_init(&k_full[b], 1);
            mbar_init(&k_empty[b], 2);            // released by both issuers
        }
        for (int b = 0; b < VS; ++b) {
            mbar_init(&v_full[b], 1);
            mbar_init(&v_empty[b], 2);            // released by both issuers
        }
        for (int r = 0; r < 2; ++r) {
            for (int h = 0; h < 2; ++h) {
                mbar_init(&s_full[r * 2 + h], 1);
                mbar_init(&p_full[r * 2 + h], 4);
                mbar_init(&pv_done[r * 2 + h], 1);
            }
        }
        mbar_fence_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp < 4) {
        setmaxnreg_dec<Regs<FP8>::kOther>();
        if (warp == 0 && lane == 0 && aligned_ok) {
            // =================================== TMA producer ================================
            tma_prefetch_desc(&tmQ);
            tma_prefetch_desc(&tmK);
            tma_prefetch_desc(&tmV);
            uint32_t it = 0;
            uint32_t q_armed = 0, k_armed = 0, v_armed = 0;   // copies started, for the drain on the way out
            bool ok = true;
            for (int si = seg_lo; si < seg_hi && ok; ++si) {
                const DevSegment seg = p.segments[si];
                if (seg.k_end <= seg.k_begin) continue;
                if (!(ok = wait_or_abort(q_empty, (q_armed & 1u) ^ 1u, ab, kWaitRingEmpty))) break;
                ++q_armed;
                mbar_expect_tx(q_full, 2 * C::TILE_BYTES);
                for (int r = 0; r < 2; ++r)
                    for (int h = 0; h < HALVES; ++h)
                        tma_load_2d(smem + C::OFF_Q + r * C::TILE_BYTES + h * HALF_BYTES, &tmQ, h * 64,
                                    seg.q_row0 + (m_tile * 2 + r) * BM, q_full);
                for (int k0 = seg.k_begin; k0 < seg.k_end; k0 += BN, ++it) {
                    const int row = seg.kv_row0 + (k0 - seg.k_begin);
                    const uint32_t kb = it % KS, kn = it / KS;
                    if (!(ok = wait_or_abort(&k_empty[kb], (kn & 1u) ^ 1u, ab, kWaitRingEmpty))) break;
                    ++k_armed;
                    if (FP8) {      // 128 keys x 128 bytes into the upper half of the stage
                        mbar_expect_tx(&k_full[kb], HALF_BYTES);
                        tma_load_2d(smem + C::OFF_K + kb * C::TILE_BYTES + HALF_BYTES, &tmK, 0, row, &k_full[kb]);
                    } else {
                        mbar_expect_tx(&k_full[kb], C::TILE_BYTES);
                        for (int h = 0; h < HALVES; ++h)
                            tma_load_2d(smem + C::OFF_K + kb * C::TILE_BYTES + h * HALF_BYTES, &tmK, h * 64, row,
                                        &k_full[kb]);
                    }
                    const uint32_t vb = it % VS, vn = it / VS;
                    if (!(ok = wait_or_abort(&v_empty[vb], (vn & 1u) ^ 1u, ab, kWaitRingEmpty))) break;
                    ++v_armed;
                    if (FP8) {
                        mbar_expect_tx(&v_full[vb], HALF_BYTES);
                        tma_load_2d(smem + C::OFF_V + vb * C::TILE_BYTES + HALF_BYTES, &tmV, 0, row, &v_full[vb]);
                    } else {
                        mbar_expect_tx(&v_full[vb], C::TILE_BYTES);
                        for (int h = 0; h < HALVES; ++h)
                            tma_load_2d(smem + C::OFF_V + vb * C::TILE_BYTES + h * HALF_BYTES, &tmV, h * 64, row,
                                        &v_full[vb]);
                    }
                }
            }
            // Every copy this thread started must have landed before the CTA may end (at once when all
            // went well: the tiles were consumed long ago).
            bool drained = q_armed == 0 || drain_wait(q_full, (q_armed - 1) & 1u, ab);
            for (uint32_t k = k_armed > (uint32_t)KS ? k_armed - KS : 0; drained && k < k_armed; ++k)
                drained = drain_wait(&k_full[k % KS], (k / KS) & 1u, ab);
            for (uint32_t k = v_armed > (uint32_t)VS ? v_armed - VS : 0; drained && k < v_armed; ++k)
                drained = drain_wait(&v_full[k % VS], (k / VS) & 1u, ab);
        } else if ((warp == 1 || warp == 2) && aligned_ok) {
            // =================================== MMA issuers =================================
            // Warp 1 + r issues every product of row tile r, half step by half step:
            //   O_r += P_r^h V^h  (key tile j)   and right behind it   S_r^h = Q_r K^h^T  (key tile j + 1).
            // The score product overwrites the buffer P_r^h sits in; the tensor pipe runs the products
            // of one thread in the order issued, so no wait (and no hand-over between two warps) is
            // needed between the two, which takes one barrier round trip out of the cycle
            // scores -> softmax -> P V -> next scores of every buffer.  The whole warp walks the
            // schedule (addresses and descriptors stay warp-uniform) and one elected lane issues:
            // issued from a diverged lane the same instructions cost several times as much.
            const int r = warp - 1;
            constexpr uint32_t idesc_qk = make_idesc(BH, false, FP8);
            constexpr uint32_t idesc_pv = make_idesc(D, true, FP8);
            const uint32_t sbase = smem_u32(smem);
            const uint32_t q_lo = desc_lo(sbase + C::OFF_Q + r * C::TILE_BYTES, 16);
            const uint32_t tmem_o = tmem_base + 2 * BN + r * BN;
            bool ok = true;
            uint32_t it = 0, n_seg = 0;

            // scores of half h of key tile `tile` (its K stage must have landed)
            auto issue_scores = [&](uint32_t tile, int h, bool last_of_segment) {
                const uint32_t kb = tile % KS;
                tc_fence_after();
                const uint32_t k_lo = desc_lo(sbase + C::OFF_K + kb * C::TILE_BYTES + h * BH * 128, 16);
                if (elect_one()) {
#pragma unroll
                    for (int ks = 0; ks < KSTEPS_QK; ++ks) {
                        const uint32_t off = ((ks >> 2) * HALF_BYTES + (ks & 3) * 32) >> 4;
                        umma_ss(tmem_base + r * BN + h * BH, desc_from_lo(q_lo + off, 1024),
                                desc_from_lo(k_lo + off, 1024), idesc_qk, ks > 0 ? 1u : 0u);
                    }
                    umma_commit(&s_full[r * 2 + h]);
                    if (h == 1) {
                        umma_commit(&k_empty[kb]);
                        if (last_of_segment) umma_commit(q_empty);   // this row tile's Q may be replaced
                    }
                }
                __syncwarp();
            };

            for (int si = seg_lo; si < seg_hi && ok; ++si) {
                const int n_tiles = (p.segments[si].k_end - p.segments[si].k_begin + BN - 1) / BN;
                if (n_tiles <= 0) continue;
                // both halves of the first key tile of the segment (its Q and K have to be there)
                if (!(ok = warp_wait(q_use, n_seg & 1u, ab, kWaitRingFull))) break;
                ++n_seg;
                if (!(ok = warp_wait(&k_use[it % KS], (it / KS) & 1u, ab, kWaitRingFull))) break;
                issue_scores(it, 0, n_tiles == 1);
                issue_scores(it, 1, n_tiles == 1);
                for (int t = 0; t < n_tiles && ok; ++t, ++it) {
                    const uint32_t vb = it % VS;
                    if (!(ok = warp_wait(&v_use[vb], (it / VS) & 1u, ab, kWaitRingFull))) break;
                    const bool more = t + 1 < n_tiles;
                    if (more && !(ok = warp_wait(&k_use[(it + 1) % KS], ((it + 1) / KS) & 1u, ab, kWaitRingFull))) break;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (!(ok = warp_wait(&p_full[r * 2 + h], it & 1u, ab, kWaitTensor))) break;
                        tc_fence_after();
                        const uint32_t v_lo = desc_lo(sbase + C::OFF_V + vb * C::TILE_BYTES + h * BH * 128, BN * 128);
                        const uint32_t a_tmem = tmem_base + r * BN + h * BH;
                        if (elect_one()) {
#pragma unroll
                            for (int ks = 0; ks < KSTEPS_PV; ++ks)
                                umma_ts(tmem_o, a_tmem + ks * 8,
                                        desc_from_lo(v_lo + ((uint32_t)(ks * 16 * 128) >> 4), 1024), idesc_pv,
                                        (t == 0 && h == 0 && ks == 0) ? 0u : 1u);
                            umma_commit(&pv_done[r * 2 + h]);
                            if (h == 1) umma_commit(&v_empty[vb]);
                        }
                        __syncwarp();
                        if (more) issue_scores(it + 1, h, t + 2 == n_tiles);
                    }
                }
            }
            // Nothing this warp issued may still be running (or still owe an arrive on one of this CTA's
            // barriers) when tensor memory is released and the CTA ends: one more commit, which
            // completes after every earlier product and commit of the issuing lane, and a wait for it.
            if (elect_one()) {
                umma_commit(&drain_bar[r]);
                drain_wait(&drain_bar[r], 0u, ab);
            }
            __syncwarp();
        }
    } else if (FP8 && warp >= 12) {
        // ======================================= widening warpgroup (8-bit cache) ============
        // Four warps, one per scheduler: the conversion instruction runs at a few lanes per clock and
        // scheduler, and one warp alone could not keep up with the tensor pipe (measured: 913 TFLOP/s on
        // the 32K-cache case with one widening warp, 1,100 with the V tiles left unwidened).  Warp w
        // handles rows 32 w .. 32 w + 31 of every tile, one row per lane.
        setmaxnreg_dec<Regs<FP8>::kWiden>();
        const int wq = warp - 12;
        if (aligned_ok) {
            // The bytes of row r were written by TMA with the 128-byte swizzle (16-byte chunk c at position
            // c ^ (r & 7)); the fp16 row goes out in the same swizzle, channels 0-63 to row r of the lower
            // half tile and 64-127 to row r of the upper one, i.e. over the bytes just read.
            auto widen_tile = [&](uint8_t* tile) {
                {
                    const int rr = wq * 32 + lane;
                    uint8_t* src = tile + HALF_BYTES + rr * 128;
                    uint4 raw[8];
#pragma unroll
                    for (int c = 0; c < 8; ++c) raw[c] = *reinterpret_cast<const uint4*>(src + ((c ^ (rr & 7)) << 4));
#pragma unroll
                    for (int c = 0; c < 8; ++c) {                 // 16 elements: channels 16 c .. 16 c + 15
                        const uint32_t w[4] = {raw[c].x, raw[c].y, raw[c].z, raw[c].w};
                        uint32_t f[8];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            f[2 * q] = e4m3x2_to_f16x2(w[q]);
                            f[2 * q + 1] = e4m3x2_to_f16x2(w[q] >> 16);
                        }
                        uint8_t* dst = tile + (c >> 2) * HALF_BYTES + rr * 128;
                        const int c0 = (c & 3) * 2;
                        *reinterpret_cast<uint4*>(dst + (((c0) ^ (rr & 7)) << 4)) = make_uint4(f[0], f[1], f[2], f[3]);
                        *reinterpret_cast<uint4*>(dst + (((c0 + 1) ^ (rr & 7)) << 4)) = make_uint4(f[4], f[5], f[6], f[7]);
                    }
                }
                fence_proxy_async_smem();                          // generic writes -> tensor core reads
                __syncwarp();
            };
            uint32_t it = 0, n_seg = 0;
            bool ok = true;
            for (int si = seg_lo; si < seg_hi && ok; ++si) {
                const int n_tiles = (p.segments[si].k_end - p.segments[si].k_begin + BN - 1) / BN;
                if (n_tiles <= 0) continue;
                // Q: bf16 -> fp16 in place (element by element, so the swizzle does not matter)
                if (!(ok = warp_wait(q_full, n_seg & 1u, ab, kWaitRingFull))) break;
                ++n_seg;
#pragma unroll 1
                for (int off = (wq * 32 + lane) * 16; off < 2 * C::TILE_BYTES; off += 128 * 16) {
                    uint4 v = *reinterpret_cast<const uint4*>(smem + C::OFF_Q + off);
                    v.x = bf16x2_to_f16x2(v.x); v.y = bf16x2_to_f16x2(v.y);
                    v.z = bf16x2_to_f16x2(v.z); v.w = bf16x2_to_f16x2(v.w);
                    *reinterpret_cast<uint4*>(smem + C::OFF_Q + off) = v;
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(q_ready);
                for (int t = 0; t < n_tiles && ok; ++t, ++it) {
                    const uint32_t kb = it % KS, vb = it % VS;
                    if (!(ok = warp_wait(&k_full[kb], (it / KS) & 1u, ab, kWaitRingFull))) break;
                    widen_tile(smem + C::OFF_K + kb * C::TILE_BYTES);
                    if (lane == 0) mbar_arrive(&k_ready[kb]);
                    if (!(ok = warp_wait(&v_full[vb], (it / VS) & 1u, ab, kWaitRingFull))) break;
                    widen_tile(smem + C::OFF_V + vb * C::TILE_BYTES);
                    if (lane == 0) mbar_arrive(&v_ready[vb]);
                }
            }
        }
    } else {
        // ======================================= softmax warpgroups ==========================
        setmaxnreg_inc<Regs<FP8>::kSoftmax>();
        const int r = (warp >> 2) - 1;                 // row tile of this warpgroup
        const int quad = warp & 3;                     // TMEM lane quadrant this warp may access
        const int row = quad * 32 + lane;              // row inside the 128-row tile
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        const uint32_t tmem_s = tmem_base + r * BN + lane_addr;
        const uint32_t tmem_o = tmem_base + 2 * BN + r * BN + lane_addr;
        const int r_local = (m_tile * 2 + r) * BM + row;   // row inside the stream's G*T rows
        const bool row_valid = r_local < p.rows_per_stream;
        uint32_t it = 0;
        bool ok = aligned_ok;

        // The exponentials of the two row tiles take turns.  The two softmax warps that share a
        // scheduler (same quadrant, row tiles 0 and 1) would otherwise run their exponentials at the
        // same time -- both are released by score products that complete back to back -- and then
        // share the special-function unit (4 results per clock and scheduler) while the rest of their
        // half step (fetch, row max, hand-overs) leaves it idle: measured, a 32-key group costs ~230
        // cycles alone and 430-500 next to its neighbour.  With turns (row tile 0, row tile 1, row tile 0,
        // ...) one warp's exponentials overlap the other's remaining work.  A turn is passed with a
        // named barrier of the two warps: the passer arrives without waiting, the taker waits.  Both
        // warps walk the same half steps, and a warp that has given up still takes and passes its
        // turns, so neither can be left waiting.
        const int bar_to_1 = 1 + quad, bar_to_0 = 5 + quad;     // barrier ids 1..8
        auto take_turn = [&](uint32_t u) {
            if (r == 1) named_barrier_sync(bar_to_1, 64);
            else if (u > 0) named_barrier_sync(bar_to_0, 64);
        };
        uint32_t turns = 0;
        auto pass_turn = [&]() {
            named_barrier_arrive(r == 0 ? bar_to_1 : bar_to_0, 64);
            ++turns;
        };
        auto skip_turn = [&](uint32_t u) {
            take_turn(u);
            pass_turn();
        };

        for (int si = seg_lo; si < seg_hi; ++si) {
            const DevSegment seg = p.segments[si];
            const int n_full = seg.n_full;     // keys visible to row 0 (row t sees n_full + t), see DevSegment
            const int n_edge = min(n_full, seg.n_kv);      // tiles that end at or below it need no mask
            const int vis = min(seg.n_kv, max(0, n_full + (r_local % p.T)));
            // sliding window: the row at position i keeps i - C < j; lo_max is the highest such bound
            const int lo = p.window > 0 ? max(0, n_full + (r_local % p.T) - p.window) : 0;
            const int lo_max = p.window > 0 ? n_full + p.T - 1 - p.window : 0;
            float m_ref = -INFINITY, l = 0.f;
            const uint32_t seg_first_it = it, seg_first_u = 2 * it;
            // 8-bit cache: the key scale of this KV head folds into the softmax scale, the value scale
            // multiplies the normalised output
            const int head = FP8 ? seg.stream % sc.Hkv : 0;
            const float scale_log2 = FP8 ? sc.score_scale_log2[head] : p.scale_log2;
            const float out_scale = FP8 ? sc.v_scale[head] : 1.f;
            for (int k0 = seg.k_begin; k0 < seg.k_end; k0 += BN, ++it) {
#pragma unroll 1
                for (int h = 0; h < 2; ++h) {
                    const uint32_t u = 2 * it + h;             // half step number
                    if (!ok) {
                        skip_turn(u);
                        continue;
                    }
                    const int kh = k0 + h * BH;                // first key of the half step
                    if (!(ok = warp_wait(&s_full[r * 2 + h], it & 1u, ab, kWaitTensor))) {
                        skip_turn(u);
                        continue;
                    }
                    tc_fence_after();
                    float s[BH];
#pragma unroll
                    for (int c = 0; c < BH / 32; ++c)
                        tmem_ld32(tmem_s + h * BH + c * 32, *reinterpret_cast<float(*)[32]>(&s[c * 32]));
                    tmem_wait_ld();

                    const bool masked = !(kh + BH <= n_edge && kh >= lo_max);   // causal edge, sequence end or window start
                    if (masked) {
#pragma unroll
                        for (int j = 0; j < BH; ++j) s[j] = (kh + j < vis && kh + j >= lo) ? s[j] : -INFINITY;
                    }
                    // row max of the raw scores (scale > 0, so it commutes with max)
                    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int j = 0; j < BH; j += 2) mx4[(j >> 1) & 3] = fmax3(mx4[(j >> 1) & 3], s[j], s[j + 1]);
                    const float mx = fmax3(fmaxf(mx4[0], mx4[1]), mx4[2], mx4[3]) * scale_log2;
                    // lazy rescale: the reference max moves only when the row max outgrew it by 2^8
                    const bool grow = mx > m_ref + kRescaleThreshold || (m_ref == -INFINITY && mx > -INFINITY);
                    if (__any_sync(0xffffffffu, grow)) {
                        float alpha = 1.f;
                        if (grow) {
                            alpha = ex2_approx(m_ref - mx);               // 0 when m_ref = -inf
                            m_ref = mx;
                            l *= alpha;
                        }
                        if (u > seg_first_u) {
                            // O_r holds the sums of the earlier half steps of this segment: wait for
                            // the product of the previous one (the other buffer; it belongs to this key
                            // tile when h = 1, to the previous one when h = 0)
                            if (!(ok = warp_wait(&pv_done[r * 2 + (h ^ 1)], (it ^ (h ^ 1)) & 1u, ab, kWaitTensor))) {
                                skip_turn(u);
                                continue;
                            }
                            tc_fence_after();
#pragma unroll 1
                            for (int c = 0; c < D / 32; ++c) {
                                float o[32];
                                tmem_ld32(tmem_o + c * 32, o);
                                tmem_wait_ld();
#pragma unroll
                                for (int j = 0; j < 32; ++j) o[j] *= alpha;
                                tmem_st32(tmem_o + c * 32, o);
                            }
                        }
                    }
                    const float neg_m = m_ref == -INFINITY ? 0.f : -m_ref;

                    // keys past the end of the sequence: their V rows may hold anything; zero them so
                    // that 0 * garbage cannot make NaN.  Both warpgroups write the same zeros in
                    // the first half step, each before it releases its own first product on this tile.
                    if (h == 0 && k0 + BN > seg.n_kv) {
                        const uint32_t vb = it % VS, vn = it / VS;
                        if (!(ok = warp_wait(&v_use[vb], vn & 1u, ab, kWaitRingFull))) {
                            skip_turn(u);
                            continue;
                        }
                        if (k0 + row >= seg.n_kv) {
                            uint8_t* vrow = smem + C::OFF_V + vb * C::TILE_BYTES + row * 128;
#pragma unroll 1
                            for (int q = 0; q < 8 * HALVES; ++q)
                                *reinterpret_cast<uint4*>(vrow + (q >> 3) * HALF_BYTES + (q & 7) * 16) = make_uint4(0u, 0u, 0u, 0u);
                        }
                        fence_proxy_async_smem();                   // generic writes -> tensor core reads
                    }

                    // P = 2^(s * scale - m_ref), two elements per instruction where the hardware
                    // allows; a masked score (-inf) comes out as exactly 0.
                    const uint64_t scale2 = f2_pack(scale_log2, scale_log2), negm2 = f2_pack(neg_m, neg_m);
                    uint64_t ls2[4] = {0ull, 0ull, 0ull, 0ull};            // packed partial row sums
                    take_turn(u);
#pragma unroll
                    for (int c = 0; c < BH / 32; ++c) {                // 32 keys -> 16 packed columns
                        uint32_t pk[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const uint64_t x2 = f2_fma(f2_pack(s[c * 32 + 2 * j], s[c * 32 + 2 * j + 1]), scale2, negm2);
                            uint64_t e2;
                            if (poly_pair(j)) {
                                e2 = f2_exp2_poly(x2);
                            } else {
                                float x0, x1;
                                f2_unpack(x2, x0, x1);
                                e2 = f2_pack(ex2_approx(x0), ex2_approx(x1));
                            }
                            ls2[j & 3] = f2_add(ls2[j & 3], e2);
                            float e0, e1;
                            f2_unpack(e2, e0, e1);
                            pk[j] = FP8 ? pack_f16x2(e0, e1) : pack_bf16x2(e0, e1);
                        }
                        tmem_st16(tmem_s + h * BH + c * 16, pk);
                    }
                    pass_turn();
                    // announce P (announcing it only after the next half step's scores had been fetched,
                    // to keep the wait for the stores out of line, was measured slower: the product
                    // that frees this buffer for the scores after next then starts later)
                    tmem_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&p_full[r * 2 + h]);
                    {
                        float a0, a1, b0, b1;
                        f2_unpack(f2_add(ls2[0], ls2[1]), a0, a1);
                        f2_unpack(f2_add(ls2[2], ls2[3]), b0, b1);
                        l += (a0 + a1) + (b0 + b1);
                    }
                }
            }
            // ---- end of segment: O_r is complete once the last PV has finished ----
            // (the products of one row tile complete in order, so the last one covers all)
            if (ok && it > seg_first_it) ok = warp_wait(&pv_done[r * 2 + 1], (it - 1) & 1u, ab, kWaitTensor);
            if (ok) {
                tc_fence_after();
                const bool has = l > 0.f;
                const float inv = has ? out_scale / l : 0.f;
                const float lse = has ? (m_ref + log2f(l)) * 0.6931471805599453f : -INFINITY;
                const bool final_out = seg.stream_nseg == 1 && !p.force_partial;
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    float o[32];
                    tmem_ld32(tmem_o + c * 32, o);
                    tmem_wait_ld();
                    if (row_valid) {
                        if (final_out) {
                            __nv_bfloat16* dst = p.O + ((int64_t)seg.q_row0 + r_local) * D + c * 32;
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                uint4 pk;
                                pk.x = pack_bf16x2(has ? o[q * 8 + 0] * inv : 0.f, has ? o[q * 8 + 1] * inv : 0.f);
                                pk.y = pack_bf16x2(has ? o[q * 8 + 2] * inv : 0.f, has ? o[q * 8 + 3] * inv : 0.f);
                                pk.z = pack_bf16x2(has ? o[q * 8 + 4] * inv : 0.f, has ? o[q * 8 + 5] * inv : 0.f);
                                pk.w = pack_bf16x2(has ? o[q * 8 + 6] * inv : 0.f, has ? o[q * 8 + 7] * inv : 0.f);
                                *reinterpret_cast<uint4*>(dst + q * 8) = pk;
                            }
                        } else {
                            float* dst = p.part_o + ((int64_t)seg.slot * p.rows_per_stream + r_local) * D + c * 32;
#pragma unroll
                            for (int q = 0; q < 8; ++q)
                                *reinterpret_cast<float4*>(dst + q * 4) =
                                    make_float4(has ? o[q * 4 + 0] * inv : 0.f, has ? o[q * 4 + 1] * inv : 0.f,
                                                has ? o[q * 4 + 2] * inv : 0.f, has ? o[q * 4 + 3] * inv : 0.f);
                        }
                    }
                }
                if (row_valid) {
                    if (final_out) {
                        if (p.lse) p.lse[seg.q_row0 + r_local] = lse;
                    } else {
                        p.part_lse[(int64_t)seg.slot * p.rows_per_stream + r_local] = lse;
                    }
                }
                tc_fence_before();
            }
        }
        // the last turn row tile 1 passed has no taker: take it, so that no barrier is left half complete
        if (r == 0 && turns > 0) named_barrier_sync(bar_to_0, 64);

    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

template <int D, bool FP8>
cudaError_t launch_one(const ChunkParams& p, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                       const CUtensorMap& tmV, int num_groups, cudaStream_t stream, const ChunkFp8Scales& sc) {
    chunk_pair_kernel<D, FP8><<<num_groups * p.m_tiles, kThreadsOf<FP8>, PCfg<D>::SMEM_BYTES, stream>>>(tmQ, tmK, tmV, p, sc);
    return cudaGetLastError();
}

template <int D, bool FP8>
cudaError_t setup_one() {
    cudaError_t e = cudaFuncSetAttribute(chunk_pair_kernel<D, FP8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         PCfg<D>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    // the register split inside the kernel assumes the launch allocation it was written for
    cudaFuncAttributes attr;
    if ((e = cudaFuncGetAttributes(&attr, chunk_pair_kernel<D, FP8>)) != cudaSuccess) return e;
    return attr.numRegs >= Regs<FP8>::kLaunch ? cudaSuccess : cudaErrorLaunchOutOfResources;
}

}  // namespace

cudaError_t chunk_pair_kernel_setup() {
    cudaError_t e = setup_one<128, false>();
    if (e != cudaSuccess) return e;
    if ((e = setup_one<64, false>()) != cudaSuccess) return e;
    return setup_one<128, true>();
}

cudaError_t launch_chunk_pair(const ChunkParams& p, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                              const CUtensorMap& tmV, int num_groups, cudaStream_t stream,
                              const ChunkFp8Scales* fp8_scales) {
    if (num_groups <= 0) return cudaSuccess;
    if (fp8_scales) {
        if (p.d != 128) return cudaErrorInvalidValue;
        return launch_one<128, true>(p, tmQ, tmK, tmV, num_groups, stream, *fp8_scales);
    }
    const ChunkFp8Scales none{};
    return p.d == 128 ? launch_one<128, false>(p, tmQ, tmK, tmV, num_groups, stream, none)
                      : launch_one<64, false>(p, tmQ, tmK, tmV, num_groups, stream, none);
}

}  // namespace yoco
