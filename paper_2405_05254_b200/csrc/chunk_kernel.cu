// Multi-token chunk / full-sequence attention on the tcgen05 tensor cores.
//
// One CTA owns one 128-row tile of the G*T query rows of a (sequence, KV head) stream and walks
// a contiguous range of 128-key tiles.  Roles (192 threads):
//   warp 0      TMA producer: Q tile once per segment, K and V tiles through two-deep rings
//   warp 1      MMA issuer (one elected lane): S = Q K^T (both operands K-major in shared memory) into one of two
//               128-column TMEM buffers, then O += P V (P K-major, V MN-major) into a third
//   warps 2..5  softmax: thread = query row; reads its S row from TMEM, keeps the running
//               max / sum, writes P (bf16) back to shared memory in the swizzled operand layout,
//               rescales O in TMEM only when the row max grew by more than 2^8, and normalises
//               and stores O (or a partial + LSE) at the end of a segment
// All shared-memory operand tiles use the 128-byte swizzle that TMA writes and the tensor-core
// descriptors read.  Every wait is bounded and reports through the status word.
#include "kernels.h"
#include "ptx.cuh"
#include "tcgen05.cuh"

namespace yoco {

namespace {

constexpr int BM = kChunkTileM;   // 128 query rows
constexpr int BN = kChunkTileN;   // 128 keys
constexpr int kThreads = 192;
constexpr int HALF_BYTES = 128 * 128;          // 128 rows x 64 bf16: one swizzled half tile
constexpr uint32_t TMEM_COLS = 512;
constexpr float kRescaleThreshold = 8.f;       // in log2 units: P stays below 2^8

template <int D>
struct CCfg {
    static constexpr int HALVES = D / 64;
    static constexpr int TILE_BYTES = HALVES * HALF_BYTES;     // Q, K or V tile
    static constexpr int P_BYTES = 2 * HALF_BYTES;             // 128 x 128 bf16
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = OFF_Q + TILE_BYTES;
    static constexpr int OFF_V = OFF_K + 2 * TILE_BYTES;
    static constexpr int OFF_P = OFF_V + 2 * TILE_BYTES;
    static constexpr int OFF_BAR = OFF_P + 2 * P_BYTES;
    static constexpr int NUM_BARS = 19;
    static constexpr int SMEM_BYTES = OFF_BAR + NUM_BARS * 8 + 16;
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
chunk_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
             const __grid_constant__ CUtensorMap tmV, const ChunkParams p) {
    using C = CCfg<D>;
    constexpr int HALVES = C::HALVES;
    constexpr int KSTEPS_QK = D / 16;
    constexpr int KSTEPS_PV = BN / 16;

    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BAR);
    uint64_t* q_full = bars + 0;
    uint64_t* q_empty = bars + 1;
    uint64_t* k_full = bars + 2;    // [2]
    uint64_t* k_empty = bars + 4;   // [2]
    uint64_t* v_full = bars + 6;    // [2]
    uint64_t* v_empty = bars + 8;   // [2]
    uint64_t* s_full = bars + 10;   // [2]
    uint64_t* s_empty = bars + 12;  // [2]
    uint64_t* p_full = bars + 14;   // [2]
    uint64_t* p_empty = bars + 16;  // [2]
    uint64_t* drain_bar = bars + 18; // everything the issuer started has finished
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
        mbar_init(q_empty, 1);
        mbar_init(drain_bar, 1);
        for (int b = 0; b < 2; ++b) {
            mbar_init(&k_full[b], 1);
            mbar_init(&k_empty[b], 1);
            mbar_init(&v_full[b], 1);
            mbar_init(&v_empty[b], 1);
            mbar_init(&s_full[b], 1);
            mbar_init(&s_empty[b], 4);
            mbar_init(&p_full[b], 4);
            mbar_init(&p_empty[b], 1);
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

    if (warp == 0) {
        // ======================================= TMA producer ================================
        if (lane == 0 && aligned_ok) {
            tma_prefetch_desc(&tmQ);
            tma_prefetch_desc(&tmK);
            tma_prefetch_desc(&tmV);
            // Two cursors walk the tiles of the group, one for K (which also brings a segment's Q, ahead of
            // its first K tile) and one for V, each as far ahead as its ring has room: the score
            // product frees a K stage long before the second product frees the V stage of the same
            // tile, and K should not wait for V.  A stage that is not free yet is looked at again on the
            // next turn; like every wait, the turns without progress are bounded.
            struct Cursor {
                int si, k0, k_end, row0;       // segment, next key, end of the segment's keys, K/V row of key 0
                bool fresh;                    // the segment's Q has not been requested yet (K cursor)
            };
            auto enter = [&](Cursor& c) {      // c.si < seg_hi: read the segment
                const DevSegment sg = p.segments[c.si];
                c.k0 = sg.k_begin;
                c.k_end = sg.k_end;
                c.row0 = sg.kv_row0 - sg.k_begin;
                c.fresh = true;
            };
            Cursor ck{seg_lo, 0, 0, 0, false}, cv{seg_lo, 0, 0, 0, false};
            if (seg_lo < seg_hi) {
                enter(ck);
                enter(cv);
            }
            uint32_t q_armed = 0, k_armed = 0, v_armed = 0;   // copies started (also for the drain on the way out)
            bool ok = true;
            uint64_t t0 = global_timer_ns();
            uint32_t idle = 0;
            while (ok && (ck.si < seg_hi || cv.si < seg_hi)) {
                bool moved = false;
                if (ck.si < seg_hi) {
                    if (ck.fresh) {            // every segment, also one without keys, gets its Q (the others wait for it)
                        if (mbar_try_wait(q_empty, (q_armed & 1u) ^ 1u)) {
                            ++q_armed;
                            mbar_expect_tx(q_full, C::TILE_BYTES);
                            for (int h = 0; h < HALVES; ++h)
                                tma_load_2d(smem + C::OFF_Q + h * HALF_BYTES, &tmQ, h * 64,
                                            p.segments[ck.si].q_row0 + m_tile * BM, q_full);
                            ck.fresh = false;
                            moved = true;
                        }
                    } else if (ck.k0 >= ck.k_end) {
                        if (++ck.si < seg_hi) enter(ck);
                        moved = true;
                    } else if (mbar_try_wait(&k_empty[k_armed & 1u], ((k_armed >> 1) & 1u) ^ 1u)) {
                        const uint32_t b = k_armed & 1u;
                        ++k_armed;
                        mbar_expect_tx(&k_full[b], C::TILE_BYTES);
                        for (int h = 0; h < HALVES; ++h)
                            tma_load_2d(smem + C::OFF_K + b * C::TILE_BYTES + h * HALF_BYTES, &tmK, h * 64, ck.row0 + ck.k0, &k_full[b]);
                        ck.k0 += BN;
                        moved = true;
                    }
                }
                if (cv.si < seg_hi) {
                    if (cv.k0 >= cv.k_end) {
                        if (++cv.si < seg_hi) enter(cv);
                        moved = true;
                    } else if (mbar_try_wait(&v_empty[v_armed & 1u], ((v_armed >> 1) & 1u) ^ 1u)) {
                        const uint32_t b = v_armed & 1u;
                        ++v_armed;
                        mbar_expect_tx(&v_full[b], C::TILE_BYTES);
                        for (int h = 0; h < HALVES; ++h)
                            tma_load_2d(smem + C::OFF_V + b * C::TILE_BYTES + h * HALF_BYTES, &tmV, h * 64, cv.row0 + cv.k0, &v_full[b]);
                        cv.k0 += BN;
                        moved = true;
                    }
                }
                if (moved) {
                    idle = 0;
                } else if ((++idle & 63u) == 0) {
                    if (idle == 64u) t0 = global_timer_ns();
                    if (*ab.flag) {
                        ok = false;
                    } else if ((int64_t)(global_timer_ns() - t0) > ab.limit_ns || idle >= kWaitMaxPolls) {
                        report_give_up(ab, kWaitRingEmpty);
                        ok = false;
                    }
                }
            }
            // Every copy this thread started must have landed before the CTA may end (at once when all
            // went well: the tiles were consumed long ago).
            bool drained = q_armed == 0 || drain_wait(q_full, (q_armed - 1) & 1u, ab);
            for (uint32_t k = k_armed > 2 ? k_armed - 2 : 0; drained && k < k_armed; ++k)
                drained = drain_wait(&k_full[k & 1u], (k >> 1) & 1u, ab);
            for (uint32_t k = v_armed > 2 ? v_armed - 2 : 0; drained && k < v_armed; ++k)
                drained = drain_wait(&v_full[k & 1u], (k >> 1) & 1u, ab);
        }
    } else if (warp == 1) {
        // ======================================= MMA issuer ==================================
        // The whole warp walks the schedule, so that addresses and descriptors stay warp-uniform;
        // one elected lane issues the tensor-core instructions.
        if (aligned_ok) {
            constexpr uint32_t idesc_qk = make_idesc(BN, false);
            constexpr uint32_t idesc_pv = make_idesc(D, true);
            const uint32_t sbase = smem_u32(smem);
            const uint64_t q_desc = make_desc(sbase + C::OFF_Q, 16, 1024);
            const uint32_t tmem_o = tmem_base + 2 * BN;
            uint32_t it = 0;
            bool ok = true;
            // PV of the previous tile is issued after QK of the current one, so that the tensor
            // pipe has work while the softmax warps process the previous S
            bool have_prev = false, prev_first = false;
            uint32_t prev_it = 0;
            auto issue_pv = [&](uint32_t i, bool first_of_segment) -> bool {
                const uint32_t b = i & 1u, n = i >> 1;
                if (!warp_wait(&p_full[b], n & 1u, ab, kWaitTensor)) return false;
                if (!warp_wait(&v_full[b], n & 1u, ab, kWaitRingFull)) return false;
                tc_fence_after();
                const uint64_t p_desc = make_desc(sbase + C::OFF_P + b * C::P_BYTES, 16, 1024);
                const uint64_t v_desc = make_desc(sbase + C::OFF_V + b * C::TILE_BYTES, BN * 128, 1024);
                if (elect_one()) {
#pragma unroll
                    for (int ks = 0; ks < KSTEPS_PV; ++ks) {
                        const uint32_t a_off = (ks >> 2) * HALF_BYTES + (ks & 3) * 32;
                        const uint32_t b_off = ks * 16 * 128;
                        umma_ss(tmem_o, p_desc + (a_off >> 4), v_desc + (b_off >> 4), idesc_pv,
                                (first_of_segment && ks == 0) ? 0u : 1u);
                    }
                    umma_commit(&p_empty[b]);
                    umma_commit(&v_empty[b]);
                }
                __syncwarp();
                return true;
            };
            for (int si = seg_lo; si < seg_hi && ok; ++si) {
                const DevSegment seg = p.segments[si];
                const uint32_t sidx = si - seg_lo;
                if (have_prev) {   // finish the previous segment before waiting for the new Q
                    if (!(ok = issue_pv(prev_it, prev_first))) break;
                    have_prev = false;
                }
                if (!(ok = warp_wait(q_full, sidx & 1u, ab, kWaitRingFull))) break;
                for (int k0 = seg.k_begin; k0 < seg.k_end; k0 += BN, ++it) {
                    const uint32_t b = it & 1u, n = it >> 1;
                    if (!(ok = warp_wait(&k_full[b], n & 1u, ab, kWaitRingFull))) break;
                    if (!(ok = warp_wait(&s_empty[b], (n & 1u) ^ 1u, ab, kWaitTensor))) break;
                    tc_fence_after();
                    const uint64_t k_desc = make_desc(sbase + C::OFF_K + b * C::TILE_BYTES, 16, 1024);
                    if (elect_one()) {
#pragma unroll
                        for (int ks = 0; ks < KSTEPS_QK; ++ks) {
                            const uint32_t off = (ks >> 2) * HALF_BYTES + (ks & 3) * 32;
                            umma_ss(tmem_base + b * BN, q_desc + (off >> 4), k_desc + (off >> 4), idesc_qk,
                                    ks > 0 ? 1u : 0u);
                        }
                        umma_commit(&s_full[b]);
                        umma_commit(&k_empty[b]);
                        if (k0 + BN >= seg.k_end) umma_commit(q_empty);   // Q may be replaced
                    }
                    __syncwarp();
                    if (have_prev && !(ok = issue_pv(prev_it, prev_first))) break;
                    have_prev = true;
                    prev_it = it;
                    prev_first = (k0 == seg.k_begin);
                }
            }
            if (ok && have_prev) issue_pv(prev_it, prev_first);
            // Nothing this warp issued may still be running (or still owe an arrive on one of this CTA's
            // barriers) when tensor memory is released and the CTA ends: one more commit, which
            // completes after every earlier product and commit of the issuing lane, and a wait for it.
            if (elect_one()) {
                umma_commit(drain_bar);
                drain_wait(drain_bar, 0u, ab);
            }
            __syncwarp();
        }
    } else {
        // ======================================= softmax warps ===============================
        const int quad = warp & 3;                     // TMEM lane quadrant this warp may access
        const int row = quad * 32 + lane;              // row inside the 128-row tile
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        const uint32_t tmem_o = tmem_base + 2 * BN + lane_addr;
        const int r_local = m_tile * BM + row;         // row inside the stream's G*T rows
        const bool row_valid = r_local < p.rows_per_stream;
        uint32_t it = 0;
        bool ok = aligned_ok;

        for (int si = seg_lo; si < seg_hi; ++si) {
            const DevSegment seg = p.segments[si];
            const int n_full = seg.n_full;     // keys visible to row 0 (row t sees n_full + t), see DevSegment
            const int n_edge = min(n_full, seg.n_kv);      // tiles that end at or below it need no mask
            const int vis = min(seg.n_kv, max(0, n_full + (r_local % p.T)));
            // sliding window: the row at position i keeps i - C < j; lo_max is the highest such bound
            const int lo = p.window > 0 ? max(0, n_full + (r_local % p.T) - p.window) : 0;
            const int lo_max = p.window > 0 ? n_full + p.T - 1 - p.window : 0;
            float m_ref = -INFINITY, l = 0.f;
            const uint32_t seg_first_it = it;

            for (int k0 = seg.k_begin; k0 < seg.k_end; k0 += BN, ++it) {
                if (!ok) continue;
                const uint32_t b = it & 1u, n = it >> 1;
                if (!(ok = warp_wait(&s_full[b], n & 1u, ab, kWaitTensor))) continue;
                tc_fence_after();
                float s[BN];
#pragma unroll
                for (int c = 0; c < BN / 32; ++c)
                    tmem_ld32(tmem_base + b * BN + lane_addr + c * 32, *reinterpret_cast<float(*)[32]>(&s[c * 32]));
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&s_empty[b]);          // S buffer may be overwritten

                // row max of the raw scores (scale > 0, so it commutes with max); four independent
                // chains keep the dependent-latency off the critical path
                if (k0 + BN > n_edge || k0 < lo_max) {   // causal edge, sequence end or window start
#pragma unroll
                    for (int j = 0; j < BN; ++j) s[j] = (k0 + j < vis && k0 + j >= lo) ? s[j] : -INFINITY;
                }
                float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                for (int j = 0; j < BN; j += 2) mx4[(j >> 1) & 3] = fmax3(mx4[(j >> 1) & 3], s[j], s[j + 1]);
                const float mx = fmax3(fmaxf(mx4[0], mx4[1]), mx4[2], mx4[3]) * p.scale_log2;
                // lazy rescale: the reference max moves only when the row max outgrew it by 2^8
                float alpha = 1.f;
                bool grow = mx > m_ref + kRescaleThreshold || (m_ref == -INFINITY && mx > -INFINITY);
                if (grow) {
                    alpha = ex2_approx(m_ref - mx);               // 0 when m_ref = -inf
                    m_ref = mx;
                    l *= alpha;
                }
                if (__any_sync(0xffffffffu, grow) && it > seg_first_it) {
                    // O holds the sums of the earlier tiles of this segment: wait for the last PV
                    const uint32_t pi = it - 1;
                    if (!(ok = warp_wait(&p_empty[pi & 1u], (pi >> 1) & 1u, ab, kWaitTensor))) continue;
                    tc_fence_after();
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        float o[32];
                        tmem_ld32(tmem_o + c * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 32; ++j) o[j] *= alpha;
                        tmem_st32(tmem_o + c * 32, o);
                    }
                    tmem_wait_st();
                    tc_fence_before();
                }
                const float m_use = m_ref == -INFINITY ? 0.f : m_ref;

                // P buffer b is free once PV of tile it-2 has completed
                if (!(ok = warp_wait(&p_empty[b], (n & 1u) ^ 1u, ab, kWaitTensor))) continue;
                uint8_t* prow = smem + C::OFF_P + b * C::P_BYTES + row * 128;
                // two elements per instruction where the hardware allows (packed fp32 multiply-add and add)
                const uint64_t scale2 = f2_pack(p.scale_log2, p.scale_log2), negm2 = f2_pack(-m_use, -m_use);
                uint64_t ls2[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
                for (int c = 0; c < BN / 8; ++c) {                 // 8 keys = one 16-byte chunk
                    uint32_t w[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        float x0, x1;
                        f2_unpack(f2_fma(f2_pack(s[c * 8 + 2 * j], s[c * 8 + 2 * j + 1]), scale2, negm2), x0, x1);
                        const float e0 = ex2_approx(x0), e1 = ex2_approx(x1);
                        ls2[j] = f2_add(ls2[j], f2_pack(e0, e1));
                        w[j] = pack_bf16x2(e0, e1);
                    }
                    *reinterpret_cast<uint4*>(prow + (c >> 3) * HALF_BYTES + (((c & 7) ^ (row & 7)) << 4)) =
                        make_uint4(w[0], w[1], w[2], w[3]);
                }
                {
                    float a0, a1, b0, b1;
                    f2_unpack(f2_add(ls2[0], ls2[1]), a0, a1);
                    f2_unpack(f2_add(ls2[2], ls2[3]), b0, b1);
                    l += (a0 + a1) + (b0 + b1);
                }

                // keys past the end of the sequence: their V rows may hold anything; zero them so
                // that 0 * garbage cannot make NaN
                if (k0 + BN > seg.n_kv) {
                    if (!(ok = warp_wait(&v_full[b], n & 1u, ab, kWaitRingFull))) continue;
                    if (k0 + row >= seg.n_kv) {
                        uint8_t* vrow = smem + C::OFF_V + b * C::TILE_BYTES + row * 128;
#pragma unroll
                        for (int h = 0; h < HALVES; ++h)
#pragma unroll
                            for (int q = 0; q < 8; ++q)
                                *reinterpret_cast<uint4*>(vrow + h * HALF_BYTES + q * 16) = make_uint4(0u, 0u, 0u, 0u);
                    }
                }
                fence_proxy_async_smem();                           // generic writes -> tensor core reads
                __syncwarp();
                if (lane == 0) mbar_arrive(&p_full[b]);
            }

            // ---- end of segment: O is complete once the last PV has finished ----
            if (ok && it > seg_first_it) {
                const uint32_t pi = it - 1;
                ok = warp_wait(&p_empty[pi & 1u], (pi >> 1) & 1u, ab, kWaitTensor);
            }
            if (ok) {
                tc_fence_after();
                const bool has = l > 0.f;
                const float inv = has ? 1.f / l : 0.f;
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
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

template <int D>
cudaError_t launch_one(const ChunkParams& p, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                       const CUtensorMap& tmV, int num_groups, cudaStream_t stream) {
    chunk_kernel<D><<<num_groups * p.m_tiles, kThreads, CCfg<D>::SMEM_BYTES, stream>>>(tmQ, tmK, tmV, p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t chunk_kernel_setup() {
    cudaError_t e = cudaFuncSetAttribute(chunk_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         CCfg<128>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(chunk_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                CCfg<64>::SMEM_BYTES);
}

cudaError_t launch_chunk(const ChunkParams& p, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                         const CUtensorMap& tmV, int num_groups, cudaStream_t stream) {
    if (num_groups <= 0) return cudaSuccess;
    return p.d == 128 ? launch_one<128>(p, tmQ, tmK, tmV, num_groups, stream)
                      : launch_one<64>(p, tmQ, tmK, tmV, num_groups, stream);
}

}  // namespace yoco
