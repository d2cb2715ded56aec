// Split-KV decode kernel: a few query rows per KV head against a long shared K/V cache.
//
// One CTA streams one contiguous range of the flat (stream, key tile) space.  A producer
// warp moves 64-key K and V tiles global -> shared with TMA (128-byte swizzle) through a
// ring of mbarrier-guarded stages; four consumer warps each take 16 keys of every tile and
// keep their own online-softmax state, so there is no CTA-wide synchronisation inside the
// key loop.  All G = Hq/Hkv query heads of the group (and the T rows of each) form the
// <= 16 rows of one mma.sync tile, so one K/V read from HBM serves the whole group.
// The arithmetic intensity is 4*G flop per K/V byte: far below the ridge, the kernel is
// bound by HBM bandwidth; the small matrix products go through mma.sync (bf16 in, fp32
// accumulate) only to keep the issue slots free for the memory pipeline.
// Row max / row sum use warp shuffles inside each quad of lanes.
//
// Work items: with p.sub_items = R > 1 every group's range is cut into R pieces (plan.h:
// sub_bound).  CTA g starts with piece 0 of group g; when its producer has issued the last
// load of an item it takes the next unclaimed one from a global counter and tells the consumer
// warps through a two-entry queue in shared memory, so the tile ring never drains between
// items.  Fast SMs thereby take more pieces than slow ones; what a piece computes and where
// its partial result goes is fixed by the plan.
#include "kernels.h"
#include "ptx.cuh"

namespace yoco {

namespace {

constexpr int kConsumerWarps = 4;
constexpr int kThreads = (kConsumerWarps + 1) * 32;
constexpr int TILE_N = kDecodeTileN;
constexpr int HALF_BYTES = TILE_N * 128;   // one 64-channel half of a tile: 64 rows x 128 B

template <int D, int ROWS>
struct Cfg {
    static constexpr int HALVES = D / 64;
    static constexpr int TENSOR_BYTES = HALVES * HALF_BYTES;
    static constexpr int STAGE_BYTES = 2 * TENSOR_BYTES;
    static constexpr int MERGE_O_BYTES = kConsumerWarps * ROWS * D * 4;
    static constexpr int MERGE_ML_BYTES = kConsumerWarps * ROWS * 2 * 4;
    // two CTAs per SM: (228 KB - 2 x 1 KB reserved) / 2 = 113 KB each
    static constexpr int BUDGET = 113 * 1024;
    static constexpr int STAGES_FIT = (BUDGET - MERGE_O_BYTES - MERGE_ML_BYTES - 128) / STAGE_BYTES;
    static constexpr int STAGES = STAGES_FIT > 4 ? 4 : STAGES_FIT;
    // + ring barriers (<= 64 B), item-queue barriers (32 B), queue entries and give-up flag
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + MERGE_O_BYTES + MERGE_ML_BYTES + 128;
    static_assert(2 * STAGES * 8 + 4 * 8 + 4 * 4 <= 128, "barrier block");
    static_assert(STAGES >= 2, "need at least a double buffer");
};

__device__ __forceinline__ uint32_t ld_global_u32(const __nv_bfloat16* p) {
    return *reinterpret_cast<const uint32_t*>(p);
}

template <int D, int ROWS>
__device__ __forceinline__ void decode_body(const CUtensorMap& tmK, const CUtensorMap& tmV,
                                            const DecodeParams& p) {
    using C = Cfg<D, ROWS>;
    constexpr int STAGES = C::STAGES;
    constexpr int KSTEPS = D / 16;
    constexpr int NT_O = D / 8;

    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* stage_mem = smem;
    float* merge_o = reinterpret_cast<float*>(smem + STAGES * C::STAGE_BYTES);
    float* merge_ml = reinterpret_cast<float*>(smem + STAGES * C::STAGE_BYTES + C::MERGE_O_BYTES);
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + STAGES * C::STAGE_BYTES +
                                                     C::MERGE_O_BYTES + C::MERGE_ML_BYTES);
    uint64_t* empty_bar = full_bar + STAGES;
    uint64_t* item_full = empty_bar + STAGES;      // [2] producer -> consumers: entry written
    uint64_t* item_empty = item_full + 2;          // [2] consumers -> producer: entry read
    volatile int32_t* item_q = reinterpret_cast<volatile int32_t*>(item_empty + 2);   // [2] item ids
    volatile int32_t* give_up = item_q + 2;        // a consumer warp ran out of patience

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int R = p.sub_items > 1 ? p.sub_items : 1;
    const int n_groups = (int)gridDim.x;
    const int n_items = n_groups * R;
    // lets a merge kernel queued behind this one be launched early; it still waits for this
    // grid to finish before it reads anything
    asm volatile("griddepcontrol.launch_dependents;");

    if ((smem_u32(smem) & 1023u) != 0) {   // the swizzle arithmetic below needs 1 KB alignment
        if (threadIdx.x == 0) atomicCAS(p.status, 0, status_word(kWaitMisaligned, linear_cta()));
        return;
    }
    const Abort ab{give_up, p.status, p.wait_limit_ns > 0 ? p.wait_limit_ns : kWaitLimitNs};
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], kConsumerWarps);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(&item_full[s], 1);
            mbar_init(&item_empty[s], kConsumerWarps);
        }
        *give_up = 0;
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
            int item = blockIdx.x;
            for (uint32_t n = 0; ok; ++n) {
                // hand the item (or the end mark) to the consumers
                if (!wait_or_abort(&item_empty[n & 1u], ((n >> 1) & 1u) ^ 1u, ab, kWaitItemQueue)) break;
                item_q[n & 1u] = item;
                mbar_arrive(&item_full[n & 1u]);
                if (item >= n_items) break;
                const int grp = item % n_groups, piece = item / n_groups;
                const int seg_lo = p.group_begin[grp], seg_hi = p.group_begin[grp + 1];
                int t_lo = 0, t_hi = 0x7fffffff, acc = 0;       // the piece's tiles inside the group
                if (R > 1) {
                    int n_g = 0;
                    for (int si = seg_lo; si < seg_hi; ++si)
                        n_g += (p.segments[si].k_end - p.segments[si].k_begin + TILE_N - 1) / TILE_N;
                    t_lo = (int)sub_bound(n_g, R, piece);
                    t_hi = (int)sub_bound(n_g, R, piece + 1);
                }
                for (int si = seg_lo; si < seg_hi && ok; ++si) {
                    const DevSegment seg = p.segments[si];
                    const int nt = (seg.k_end - seg.k_begin + TILE_N - 1) / TILE_N;
                    const int s_lo = max(t_lo - acc, 0), s_hi = min(t_hi - acc, nt);
                    acc += nt;
                    if (s_lo >= s_hi) continue;
                    const int k_lo = seg.k_begin + s_lo * TILE_N;
                    const int k_hi = min(seg.k_begin + s_hi * TILE_N, seg.k_end);
                    for (int k0 = k_lo; k0 < k_hi; k0 += TILE_N, ++it) {
                        const uint32_t stage = it % STAGES, round = it / STAGES;
                        // self-test of the give-up path: nothing is armed, so no stage is needed either
                        // and the wait that runs out is the consumers' first wait for a tile
                        if (p.selftest_skip_loads) continue;
                        if (!wait_or_abort(&empty_bar[stage], (round & 1u) ^ 1u, ab, kWaitRingEmpty)) {
                            ok = false;
                            break;
                        }
                        uint8_t* kdst = stage_mem + stage * C::STAGE_BYTES;
                        uint8_t* vdst = kdst + C::TENSOR_BYTES;
                        mbar_expect_tx(&full_bar[stage], C::STAGE_BYTES);
                        const int row = seg.kv_row0 + (k0 - seg.k_begin);
#pragma unroll
                        for (int h = 0; h < C::HALVES; ++h) {
                            tma_load_2d(kdst + h * HALF_BYTES, &tmK, h * 64, row, &full_bar[stage]);
                            tma_load_2d(vdst + h * HALF_BYTES, &tmV, h * 64, row, &full_bar[stage]);
                        }
                    }
                }
                // all loads of this item are on their way: claim the next one
                item = R > 1 ? n_groups + atomicAdd(p.work_counter, 1) : n_items;
            }
            // Before this thread leaves, every copy it armed must have landed: the CTA ends when its
            // last thread does, and a copy that lands later would write into (and arrive on barriers
            // in) shared memory that already belongs to another CTA.  When all went well the
            // consumers are still reading these tiles and the waits return at once.
            if (!p.selftest_skip_loads) {
                const uint32_t in_flight = it < (uint32_t)STAGES ? it : (uint32_t)STAGES;
                for (uint32_t k = it - in_flight; k < it; ++k)
                    if (!drain_wait(&full_bar[k % STAGES], (k / STAGES) & 1u, ab)) break;
            }
        }
        return;
    }

    // ----------------------------------- consumers ---------------------------------------
    const int g = lane >> 2, tq = lane & 3;
    const int n_rows = p.rows_per_stream;
    uint32_t it = 0;
    bool ok = true;

    for (uint32_t n_item = 0;; ++n_item) {
        // the next item from the producer; the four warps must take the same decision, so a warp
        // that gives up waiting says so before the barrier and all of them leave together
        const bool got_item = wait_or_abort(&item_full[n_item & 1u], (n_item >> 1) & 1u, ab, kWaitItemQueue);
        const int item = item_q[n_item & 1u];
        // one answer for all four warps (a barrier that ORs): nobody reads the flag on its own
        if (named_barrier_or(1, kConsumerWarps * 32, !got_item || !ok)) break;
        if (lane == 0) mbar_arrive(&item_empty[n_item & 1u]);
        if (item >= n_items) break;
        const int grp = item % n_groups, piece = item / n_groups;
        const int seg_lo = p.group_begin[grp], seg_hi = p.group_begin[grp + 1];
        int t_lo = 0, t_hi = 0x7fffffff, t_acc = 0;       // the piece's tiles inside the group
        if (R > 1) {
            int n_g = 0;
            for (int si = seg_lo; si < seg_hi; ++si)
                n_g += (p.segments[si].k_end - p.segments[si].k_begin + TILE_N - 1) / TILE_N;
            t_lo = (int)sub_bound(n_g, R, piece);
            t_hi = (int)sub_bound(n_g, R, piece + 1);
        }

        for (int si = seg_lo; si < seg_hi; ++si) {
            const DevSegment seg = p.segments[si];
            const int seg_tiles = (seg.k_end - seg.k_begin + TILE_N - 1) / TILE_N;
            const int s_lo = max(t_lo - t_acc, 0), s_hi = min(t_hi - t_acc, seg_tiles);
            t_acc += seg_tiles;
            const int slot = seg.slot * R + piece;
            if (s_lo >= s_hi) {
                // this piece holds nothing of the segment: its slot must say so to the merge
                if (R > 1 && threadIdx.x < n_rows) p.part_lse[(int64_t)slot * n_rows + threadIdx.x] = -INFINITY;
                continue;
            }
            const int k_lo = seg.k_begin + s_lo * TILE_N;
            const int k_hi = min(seg.k_begin + s_hi * TILE_N, seg.k_end);

            // Q as the A operand of m16n8k16: rows = (head in group, t), zero beyond n_rows
            uint32_t qa[KSTEPS][4];
            {
                const __nv_bfloat16* q0 = p.Q + ((int64_t)seg.q_row0 + g) * D + tq * 2;
                const __nv_bfloat16* q1 = q0 + 8 * D;
                const bool v0 = g < n_rows, v1 = ROWS == 16 && (g + 8) < n_rows;
#pragma unroll
                for (int ks = 0; ks < KSTEPS; ++ks) {
                    qa[ks][0] = v0 ? ld_global_u32(q0 + ks * 16) : 0u;
                    qa[ks][1] = v1 ? ld_global_u32(q1 + ks * 16) : 0u;
                    qa[ks][2] = v0 ? ld_global_u32(q0 + ks * 16 + 8) : 0u;
                    qa[ks][3] = v1 ? ld_global_u32(q1 + ks * 16 + 8) : 0u;
                }
            }
            // causal limits: row t sees keys j < n_full + t (n_full = N - T + 1 for a whole cache; for a key
            // shard the same count less the keys of earlier shards) and none past the keys held here
            const int n_full = seg.n_full;
            const int n_edge = min(n_full, seg.n_kv);      // tiles that end at or below it need no mask
            const int vis0 = min(seg.n_kv, max(0, n_full + (g % p.T)));
            const int vis1 = min(seg.n_kv, max(0, n_full + ((g + 8) % p.T)));

            float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
            float o[NT_O][4];
#pragma unroll
            for (int nt = 0; nt < NT_O; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;

            for (int k0 = k_lo; k0 < k_hi; k0 += TILE_N, ++it) {
                if (!ok) continue;
                const uint32_t stage = it % STAGES, round = it / STAGES;
                if (!wait_or_abort(&full_bar[stage], round & 1u, ab, kWaitRingFull)) {
                    ok = false;     // this warp touches no tile any more; it still walks to the barriers below
                    continue;
                }
                const int kw = k0 + warp * 16;          // first key of this warp's slice
                if (kw < k_hi) {
                    const uint32_t kbase = smem_u32(stage_mem + stage * C::STAGE_BYTES);
                    const uint32_t vbase = kbase + C::TENSOR_BYTES;

                    // ---- S = Q K^T for 16 keys (two n-tiles of 8 keys) ----
                    float s[2][4];
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
                    {
                        const int key_l = warp * 16 + (lane >> 4) * 8 + (lane & 7);
                        const int sel = (lane >> 3) & 1;
                        const uint32_t rowaddr = kbase + key_l * 128;
#pragma unroll
                        for (int ks = 0; ks < KSTEPS; ++ks) {
                            const int c = 2 * ks + sel;
                            const uint32_t addr =
                                rowaddr + (c >> 3) * HALF_BYTES + ((((c & 7) ^ key_l) & 7) << 4);
                            uint32_t b0, b1, b2, b3;
                            ldmatrix_x4(addr, b0, b1, b2, b3);
                            mma_bf16_16816(s[0], qa[ks], b0, b1);
                            mma_bf16_16816(s[1], qa[ks], b2, b3);
                        }
                    }
                    // ---- scale, mask, online softmax ----
                    // sliding window: the row at position i keeps i - C < j, i.e. j >= i - C + 1 =
                    // n_full + t - C; the highest such bound of any row is n_full + T - 1 - C
                    const bool need_mask = kw + 16 > n_edge || (p.window > 0 && kw < n_full + p.T - 1 - p.window);
                    // window start of the two rows this lane holds (no window: below every key)
                    int lo0 = -1, lo1 = -1;
                    if (need_mask && p.window > 0) {
                        lo0 = n_full + (g % p.T) - p.window;
                        lo1 = n_full + ((g + 8) % p.T) - p.window;
                    }
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            float v = s[nt][e] * p.scale_log2;
                            if (need_mask) {
                                const int j = kw + nt * 8 + tq * 2 + (e & 1);
                                v = (j < ((e & 2) ? vis1 : vis0) && j >= ((e & 2) ? lo1 : lo0)) ? v : -INFINITY;
                            }
                            s[nt][e] = v;
                        }
                    float mx0 = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
                    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
                    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
                    const float mn0 = fmaxf(m0, mx0);
                    const float ms0 = mn0 == -INFINITY ? 0.f : mn0;
                    const float alpha0 = exp2f(m0 - ms0);
                    m0 = mn0;
                    float alpha1 = 1.f, ms1 = 0.f;
                    if (ROWS == 16) {
                        float mx1 = fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]));
                        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
                        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
                        const float mn1 = fmaxf(m1, mx1);
                        ms1 = mn1 == -INFINITY ? 0.f : mn1;
                        alpha1 = exp2f(m1 - ms1);
                        m1 = mn1;
                    }
                    uint32_t pa[4];
                    {
                        const float p00 = exp2f(s[0][0] - ms0), p01 = exp2f(s[0][1] - ms0);
                        const float p10 = exp2f(s[1][0] - ms0), p11 = exp2f(s[1][1] - ms0);
                        l0 = l0 * alpha0 + ((p00 + p01) + (p10 + p11));
                        pa[0] = pack_bf16x2(p00, p01);
                        pa[2] = pack_bf16x2(p10, p11);
                        if (ROWS == 16) {
                            const float q00 = exp2f(s[0][2] - ms1), q01 = exp2f(s[0][3] - ms1);
                            const float q10 = exp2f(s[1][2] - ms1), q11 = exp2f(s[1][3] - ms1);
                            l1 = l1 * alpha1 + ((q00 + q01) + (q10 + q11));
                            pa[1] = pack_bf16x2(q00, q01);
                            pa[3] = pack_bf16x2(q10, q11);
                        } else {
                            pa[1] = pa[3] = 0u;
                        }
                    }
                    if (__any_sync(0xffffffffu, alpha0 != 1.f || alpha1 != 1.f)) {
#pragma unroll
                        for (int nt = 0; nt < NT_O; ++nt) {
                            o[nt][0] *= alpha0; o[nt][1] *= alpha0;
                            o[nt][2] *= alpha1; o[nt][3] *= alpha1;
                        }
                    }
                    // ---- rows past the end of the sequence may hold anything: zero them so that
                    //      0 * garbage cannot produce NaN in O += P V ----
                    if (kw + 16 > seg.n_kv) {
                        const int first_bad = max(seg.n_kv - kw, 0);          // 0..15
                        uint8_t* vrow = stage_mem + stage * C::STAGE_BYTES + C::TENSOR_BYTES;
                        for (int r = first_bad; r < 16; ++r) {
                            const int key_l = warp * 16 + r;
                            for (int b = lane * 16; b < C::HALVES * 128; b += 512) {
                                const int h = b >> 7, off = b & 127;
                                *reinterpret_cast<uint4*>(vrow + h * HALF_BYTES + key_l * 128 + off) =
                                    make_uint4(0u, 0u, 0u, 0u);
                            }
                        }
                        __syncwarp();
                    }
                    // ---- O += P V ----
                    {
                        const int key_l = warp * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
                        const int sel = lane >> 4;
                        const uint32_t rowaddr = vbase + key_l * 128;
#pragma unroll
                        for (int nt = 0; nt < NT_O; nt += 2) {
                            const int c = nt + sel;
                            const uint32_t addr =
                                rowaddr + (c >> 3) * HALF_BYTES + ((((c & 7) ^ key_l) & 7) << 4);
                            uint32_t b0, b1, b2, b3;
                            ldmatrix_x4_trans(addr, b0, b1, b2, b3);
                            mma_bf16_16816(o[nt], pa, b0, b1);
                            mma_bf16_16816(o[nt + 1], pa, b2, b3);
                        }
                    }
                    if (kw + 16 > seg.n_kv) fence_proxy_async_smem();   // generic writes before TMA reuse
                }
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
                float* mo = merge_o + (warp * ROWS) * D;
#pragma unroll
                for (int nt = 0; nt < NT_O; ++nt) {
                    *reinterpret_cast<float2*>(mo + g * D + nt * 8 + tq * 2) = make_float2(o[nt][0], o[nt][1]);
                    if (ROWS == 16)
                        *reinterpret_cast<float2*>(mo + (g + 8) * D + nt * 8 + tq * 2) =
                            make_float2(o[nt][2], o[nt][3]);
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
            const bool final_out = seg.stream_nseg == 1 && !p.force_partial && R == 1;
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
                const float outv = L > 0.f ? acc / L : 0.f;
                const float lse = L > 0.f ? (M + log2f(L)) * 0.6931471805599453f : -INFINITY;
                if (final_out) {
                    p.O[((int64_t)seg.q_row0 + r) * D + col] = __float2bfloat16(outv);
                    if (p.lse && col == 0) p.lse[seg.q_row0 + r] = lse;
                } else {
                    p.part_o[((int64_t)slot * n_rows + r) * D + col] = outv;
                    if (col == 0) p.part_lse[(int64_t)slot * n_rows + r] = lse;
                }
            }
            named_barrier_sync(1, kConsumerWarps * 32);
        }
    }
}

// work tables in global memory (the workspace)
template <int D, int ROWS>
__global__ void __launch_bounds__(kThreads, 2)
decode_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
              const DecodeParams p) {
    decode_body<D, ROWS>(tmK, tmV, p);
}

// work tables as kernel parameters
template <int D, int ROWS>
__global__ void __launch_bounds__(kThreads, 2)
decode_kernel_inline(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                     const DecodeParams p0, const __grid_constant__ DecodeInlineTables tab) {
    DecodeParams p = p0;
    p.segments = tab.seg;
    p.group_begin = tab.group_begin;
    decode_body<D, ROWS>(tmK, tmV, p);
}

template <int D, int ROWS>
cudaError_t launch_one(const DecodeParams& p, const CUtensorMap& tmK, const CUtensorMap& tmV,
                       int num_groups, cudaStream_t stream, const DecodeInlineTables* inline_tab) {
    using C = Cfg<D, ROWS>;
    if (inline_tab)
        decode_kernel_inline<D, ROWS><<<num_groups, kThreads, C::SMEM_BYTES, stream>>>(tmK, tmV, p, *inline_tab);
    else
        decode_kernel<D, ROWS><<<num_groups, kThreads, C::SMEM_BYTES, stream>>>(tmK, tmV, p);
    return cudaGetLastError();
}

template <int D, int ROWS>
cudaError_t setup_one() {
    cudaError_t e = cudaFuncSetAttribute(decode_kernel<D, ROWS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         Cfg<D, ROWS>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(decode_kernel_inline<D, ROWS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                Cfg<D, ROWS>::SMEM_BYTES);
}

}  // namespace

cudaError_t decode_kernel_setup() {
    cudaError_t e;
    if ((e = setup_one<128, 8>()) != cudaSuccess) return e;
    if ((e = setup_one<128, 16>()) != cudaSuccess) return e;
    if ((e = setup_one<64, 8>()) != cudaSuccess) return e;
    return setup_one<64, 16>();
}

cudaError_t launch_decode(const DecodeParams& p, const CUtensorMap& tmK, const CUtensorMap& tmV,
                          int num_groups, cudaStream_t stream, const DecodeInlineTables* tab) {
    if (num_groups <= 0) return cudaSuccess;
    const bool wide = p.rows_per_stream > 8;
    if (p.d == 128)
        return wide ? launch_one<128, 16>(p, tmK, tmV, num_groups, stream, tab)
                    : launch_one<128, 8>(p, tmK, tmV, num_groups, stream, tab);
    return wide ? launch_one<64, 16>(p, tmK, tmV, num_groups, stream, tab)
                : launch_one<64, 8>(p, tmK, tmV, num_groups, stream, tab);
}

}  // namespace yoco
