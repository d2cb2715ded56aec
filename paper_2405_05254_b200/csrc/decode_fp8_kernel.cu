// Split-KV decode over an 8-bit cache: K and V stored as FP8 E4M3 bytes with one fp32 scale per
// KV head (value = scale[c] * e4m3(byte)), head dimension 128.  Same structure as the bf16 decode
// kernel (one CTA per contiguous range of the flat (stream, key tile) space, a TMA producer warp,
// four consumer warps with their own online-softmax state), but a 64-key tile is 8 KB per tensor,
// so the same HBM bandwidth streams twice as many keys, and each consumer warp takes whole tiles
// in turn (instead of a quarter of every tile) so that its fixed latencies are paid per 64 keys.
//
// The bytes are widened to fp16 in registers (cvt.rn.f16x2.e4m3x2 is exact) and the small
// products run as m16n8k16 fp16 MMAs with fp32 accumulation; Q is converted bf16 -> fp16 once per
// segment and P is rounded to fp16.  With at most 16 query rows per stream the products are taken
// transposed, keys and channels on the 16-wide side of the instruction:
//   S^T (keys x rows)     = K (keys x channels)      Q^T
//   O^T (channels x rows) = V^T (channels x keys)    P^T
// so that no tensor-core row is padding when there are 8 rows or fewer: half the products of the
// rows-on-the-16-side form, and these warp-level products are what a consumer warp spends most of
// its time on (measured: the same kernel with half the products issued ran 6 % faster, while
// removing two fifths of its other instructions changed nothing).  P^T comes out of the score
// product with a key per lane group and has to become an operand with a query row per lane group: one
// movmatrix (8 x 8 transpose of 16-bit units) per 8 keys.  Because ldmatrix moves 16-bit units, a lane
// receives four consecutive channels of a key (K) or two channels of two consecutive keys (V,
// transposed); the reduction index of a product may be permuted freely as long as both operands
// agree, and so may the order of the output channels: Q is loaded with the matching channel order
// and the output channels are put back in order when the accumulators are written out.  The
// scales multiply the scores (k_scale, folded into the softmax scale) and the output (v_scale).
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
    static constexpr int STAGES_FIT = (BUDGET - MERGE_O_BYTES - MERGE_ML_BYTES - 256) / STAGE_BYTES;
    static constexpr int STAGES = STAGES_FIT > 6 ? 6 : STAGES_FIT;
    static_assert(STAGES >= kConsumerWarps, "every consumer warp needs a tile in flight");
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + MERGE_O_BYTES + MERGE_ML_BYTES + 256;
    static_assert(STAGES >= 2, "need at least a double buffer");
};

// D(16x8, f32) += A(16x16, f16, row) * B(16x8, f16, col)
__device__ __forceinline__ void mma_f16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// 8 x 8 transpose of 16-bit units across the warp: lane (g, tq) gives row g, columns 2 tq and 2 tq + 1,
// and receives the same positions of the transposed matrix.
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
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
__device__ __forceinline__ float ex2_fast(float x) {   // 2^x, one special-function op; 2^-inf = 0
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ void st_release_shared(uint32_t* p, uint32_t v) {
    asm volatile("st.release.cta.shared::cta.u32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire_shared(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.cta.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)) : "memory");
    return v;
}
// Waits (bounded, like every wait) until the producer's count of armed tiles has reached `want`.
__device__ __forceinline__ bool wait_armed(const uint32_t* armed, uint32_t want, const Abort& ab) {
    if (ld_acquire_shared(armed) >= want) return true;
    const uint64_t t0 = global_timer_ns();
    for (uint32_t i = 1;; ++i) {
        if (ld_acquire_shared(armed) >= want) return true;
        if ((i & 63u) == 0) {
            if (*ab.flag) return false;
            if ((int64_t)(global_timer_ns() - t0) > ab.limit_ns || i >= kWaitMaxPolls) {
                report_give_up(ab, kWaitItemQueue);
                return false;
            }
        }
    }
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
    uint32_t* armed = reinterpret_cast<uint32_t*>(empty_bar + STAGES) + 1;         // tiles the producer has armed so far
    uint64_t* item_full = empty_bar + STAGES + 1;  // [2] producer -> consumers: queue entry written
    uint64_t* item_empty = item_full + 2;          // [2] consumers -> producer: entry read
    volatile int32_t* item_q = reinterpret_cast<volatile int32_t*>(item_empty + 2);   // [2] item ids
    static_assert(2 * STAGES * 8 + 8 + 32 + 8 <= 256, "barrier block");

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Work items as in the bf16 kernel: with R = p.sub_items > 1 every group's range is cut into R
    // pieces; CTA g starts with piece 0 of group g and its producer, once the last copy of an item
    // is on its way, claims the next unclaimed piece from a global counter and tells the consumers
    // through a two-entry queue, so that the ring never drains between items and a fast SM takes
    // more pieces than a slow one.  What a piece computes and where its partial result goes is
    // fixed by the plan.
    const int R = p.sub_items > 1 ? p.sub_items : 1;
    const int n_groups = gridDim.x;
    const int n_items = n_groups * R;
    asm volatile("griddepcontrol.launch_dependents;");

    if ((smem_u32(smem) & 1023u) != 0) {   // the swizzle arithmetic below needs 1 KB alignment
        if (threadIdx.x == 0) atomicCAS(p.status, 0, status_word(kWaitMisaligned, linear_cta()));
        return;
    }
    const Abort ab{give_up, p.status, p.wait_limit_ns > 0 ? p.wait_limit_ns : kWaitLimitNs};
    if (threadIdx.x == 0) {
        *give_up = 0;
        *armed = 0u;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);                 // released by the one warp that read the tile
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(&item_full[s], 1);
            mbar_init(&item_empty[s], kConsumerWarps);
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
            int item = blockIdx.x;
            for (uint32_t n = 0; ok; ++n) {
                // hand the item (or the end mark) to the consumers
                if (!wait_or_abort(&item_empty[n & 1u], ((n >> 1) & 1u) ^ 1u, ab, kWaitItemQueue)) break;
                item_q[n & 1u] = item;
                mbar_arrive(&item_full[n & 1u]);
                if (item >= n_items) break;
                const int grp = item % n_groups, piece = item / n_groups;
                const int seg_lo = group_begin[grp], seg_hi = group_begin[grp + 1];
                int t_lo = 0, t_hi = 0x7fffffff, t_acc = 0;     // the piece's tiles inside the group
                if (R > 1) {
                    int n_g = 0;
                    for (int si = seg_lo; si < seg_hi; ++si)
                        n_g += (segments[si].k_end - segments[si].k_begin + TILE_N - 1) / TILE_N;
                    t_lo = (int)sub_bound(n_g, R, piece);
                    t_hi = (int)sub_bound(n_g, R, piece + 1);
                }
                for (int si = seg_lo; si < seg_hi && ok; ++si) {
                    const DevSegment seg = segments[si];
                    const int seg_tiles = (seg.k_end - seg.k_begin + TILE_N - 1) / TILE_N;
                    const int s_lo = max(t_lo - t_acc, 0), s_hi = min(t_hi - t_acc, seg_tiles);
                    t_acc += seg_tiles;
                    if (s_lo >= s_hi) continue;
                    const int k_lo = seg.k_begin + s_lo * TILE_N;
                    const int k_hi = min(seg.k_begin + s_hi * TILE_N, seg.k_end);
                    for (int k0 = k_lo; k0 < k_hi; k0 += TILE_N, ++it) {
                        const uint32_t stage = it % STAGES, round = it / STAGES;
                        // self-test of the give-up path: nothing is armed, so no stage is needed either and
                        // the wait that runs out is the consumers' wait for the producer to arm their tile
                        if (p.selftest_skip_loads) continue;
                        if (!wait_or_abort(&empty_bar[stage], (round & 1u) ^ 1u, ab, kWaitRingEmpty)) {
                            ok = false;
                            break;
                        }
                        uint8_t* kdst = stage_mem + stage * STAGE_BYTES;
                        mbar_expect_tx(&full_bar[stage], STAGE_BYTES);
                        const int row = seg.kv_row0 + (k0 - seg.k_begin);
                        tma_load_2d(kdst, &tmK, 0, row, &full_bar[stage]);
                        tma_load_2d(kdst + TENSOR_BYTES, &tmV, 0, row, &full_bar[stage]);
                        st_release_shared(armed, it + 1);        // tiles 0 .. it have their barriers armed
                    }
                }
                // all loads of this item are on their way: claim the next one
                item = R > 1 ? n_groups + atomicAdd(p.work_counter, 1) : n_items;
            }
            // every copy this thread armed must have landed before it leaves (the CTA ends with its last
            // thread, and its shared memory then belongs to another CTA); at once when all went well
            if (!p.selftest_skip_loads) {
                const uint32_t in_flight = it < (uint32_t)STAGES ? it : (uint32_t)STAGES;
                for (uint32_t k = it - in_flight; k < it; ++k)
                    if (!drain_wait(&full_bar[k % STAGES], (k / STAGES) & 1u, ab)) break;
            }
        }
        return;
    }

    // ----------------------------------- consumers ---------------------------------------
    // Each consumer warp takes WHOLE tiles, round robin (tile number mod 4): per tile a warp then runs
    // one softmax for 64 keys instead of one per 16, which matters here because at half the bytes
    // per key the chain of dependent latencies per tile (products, shuffles, exponentials), not
    // the memory, would otherwise set the pace.  A tile is released by the one warp that read it.
    constexpr int NT = ROWS / 8;                       // 8-row groups on the narrow side of the products
    const int g = lane >> 2, tq = lane & 3;
    const int n_rows = p.rows_per_stream;
    // row address this lane supplies to ldmatrix.x4 for K: matrix (lane >> 3) = (16-byte chunk of the pair, key half)
    const int ld_key16 = ((lane >> 3) & 1) * 8 + (lane & 7);            // key row inside a 16-key group
    const int ld_chunk = lane >> 4;                                      // 0: first chunk of the pair, 1: second
    uint32_t it = 0;
    bool ok = true;

    for (uint32_t n_item = 0;; ++n_item) {
    // the next item from the producer; the four warps must take the same decision, so a warp
    // that gives up waiting says so before the barrier and all of them leave together
    const bool got_item = wait_or_abort(&item_full[n_item & 1u], (n_item >> 1) & 1u, ab, kWaitItemQueue);
    const int item = item_q[n_item & 1u];
    if (named_barrier_or(1, kConsumerWarps * 32, !got_item || !ok)) break;
    if (lane == 0) mbar_arrive(&item_empty[n_item & 1u]);
    if (item >= n_items) break;
    const int grp = item % n_groups, piece = item / n_groups;
    const int seg_lo = group_begin[grp], seg_hi = group_begin[grp + 1];
    int t_lo = 0, t_hi = 0x7fffffff, t_acc = 0;       // the piece's tiles inside the group
    if (R > 1) {
        int n_g = 0;
        for (int si = seg_lo; si < seg_hi; ++si)
            n_g += (segments[si].k_end - segments[si].k_begin + TILE_N - 1) / TILE_N;
        t_lo = (int)sub_bound(n_g, R, piece);
        t_hi = (int)sub_bound(n_g, R, piece + 1);
    }

    for (int si = seg_lo; si < seg_hi; ++si) {
        const DevSegment seg = segments[si];
        const int seg_tiles = (seg.k_end - seg.k_begin + TILE_N - 1) / TILE_N;
        const int s_lo = max(t_lo - t_acc, 0), s_hi = min(t_hi - t_acc, seg_tiles);
        t_acc += seg_tiles;
        const int slot = seg.slot * R + piece;
        if (s_lo >= s_hi) {
            // this piece holds nothing of the segment: its slot must say so to the merge
            if (R > 1 && threadIdx.x < p.rows_per_stream) p.part_lse[(int64_t)slot * p.rows_per_stream + threadIdx.x] = -INFINITY;
            continue;
        }
        const int k_lo = seg.k_begin + s_lo * TILE_N;
        const int k_hi = min(seg.k_begin + s_hi * TILE_N, seg.k_end);
        const int head = seg.stream % pp.Hkv;
        const float sscale = pp.score_scale_log2[head], vscale = pp.v_scale[head];

        // Q^T as the second operand of the score product (fp16).  Reduction step ks covers channels
        // 16 ks .. 16 ks + 15, and this lane's four reduction slots (k = 2 tq, 2 tq + 1, 2 tq + 8, 2 tq + 9)
        // stand for the four consecutive channels 16 ks + 4 tq + {0, 1, 2, 3} of query row 8 nt + g: the
        // order in which ldmatrix hands it K bytes.
        uint32_t qb[NT][8][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int row = 8 * nt + g;
            const __nv_bfloat16* q = p.Q + ((int64_t)seg.q_row0 + row) * D + tq * 4;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const uint2 w = row < n_rows ? *reinterpret_cast<const uint2*>(q + ks * 16) : make_uint2(0u, 0u);
                qb[nt][ks][0] = pack_f16x2(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xFFFF0000u));
                qb[nt][ks][1] = pack_f16x2(__uint_as_float(w.y << 16), __uint_as_float(w.y & 0xFFFF0000u));
            }
        }
        const int n_full = seg.n_full;
        const int n_edge = min(n_full, seg.n_kv);      // tiles that end at or below it need no mask
        int vis[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) vis[nt][e] = min(seg.n_kv, max(0, n_full + ((8 * nt + 2 * tq + e) % p.T)));

        // running max and (this lane's part of the) sum of rows 8 nt + 2 tq + {0, 1}
        float m[NT][2], l[NT][2];
        // O^T: acc[nt][j][e] is the product tile whose channel slot i stands for channel 32 j + 2 i + e
        // (i < 8) or 32 j + 16 + 2 (i - 8) + e: elements 0, 1 = (slot g, rows 2 tq, 2 tq + 1), elements
        // 2, 3 = (slot g + 8, same rows)
        float acc[NT][4][2][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            m[nt][0] = m[nt][1] = -INFINITY;
            l[nt][0] = l[nt][1] = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int e = 0; e < 2; ++e) acc[nt][j][e][0] = acc[nt][j][e][1] = acc[nt][j][e][2] = acc[nt][j][e][3] = 0.f;
        }

        for (int k0 = k_lo; k0 < k_hi; k0 += TILE_N, ++it) {
            if (!ok || (int)(it % kConsumerWarps) != warp) continue;       // not this warp's tile
            // A parity wait only tells the phase of a barrier apart from the one before it.  A warp
            // that takes every fourth tile could ask for round r of a stage whose round r - 1 has not
            // landed yet (copies complete in any order, and when a kernel starts all of them queue at
            // once): it would be let through at once, read a tile that is still being written and
            // release the stage a second time.  So it first waits until the producer has armed
            // THIS tile: the producer can only have done so after the previous tile of the stage was
            // released, i.e. after its round completed, and the barrier is then in the round asked for.
            const uint32_t stage = it % STAGES, round = it / STAGES;
            if (!wait_armed(armed, it + 1, ab) || !wait_or_abort(&full_bar[stage], round & 1u, ab, kWaitRingFull)) {
                ok = false;         // this warp touches no tile any more; it still walks to the barriers below
                continue;
            }
            const uint32_t kbase = smem_u32(stage_mem + stage * STAGE_BYTES);
            const uint32_t vbase = kbase + TENSOR_BYTES;

            // ---- S^T = K Q^T for 64 keys: four 16-key groups, eight 16-channel reduction steps.
            //      (The key groups of a step are fetched first and their products issued side by
            //      side: products into the same accumulator wait for one another.) ----
            float s[NT][4][4];     // [row group][16-key group]: (key g, rows 2 tq, 2 tq + 1), (key g + 8, same rows)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int mt = 0; mt < 4; ++mt) s[nt][mt][0] = s[nt][mt][1] = s[nt][mt][2] = s[nt][mt][3] = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int chunk = 2 * j + ld_chunk;
                uint32_t r[4][4];   // per key group: (keys 0-7, chunk 2 j) (keys 8-15, 2 j) (keys 0-7, 2 j + 1) (keys 8-15, 2 j + 1)
#pragma unroll
                for (int mt = 0; mt < 4; ++mt) {
                    const int key = mt * 16 + ld_key16;
                    ldmatrix_x4(kbase + key * 128 + (((chunk ^ key) & 7) << 4), r[mt][0], r[mt][1], r[mt][2], r[mt][3]);
                }
#pragma unroll
                for (int h = 0; h < 2; ++h)                // chunk 2 j + h = reduction step ks
#pragma unroll
                    for (int mt = 0; mt < 4; ++mt) {
                        const uint32_t lo = r[mt][2 * h], hi = r[mt][2 * h + 1];     // key g, key g + 8
                        const uint32_t a0 = e4m3x2_to_f16x2(lo), a2 = e4m3x2_to_f16x2(lo >> 16);
                        const uint32_t a1 = e4m3x2_to_f16x2(hi), a3 = e4m3x2_to_f16x2(hi >> 16);
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt)
                            mma_f16_16816(s[nt][mt], a0, a1, a2, a3, qb[nt][2 * j + h][0], qb[nt][2 * j + h][1]);
                    }
            }
            // ---- scale, mask (causal edge, sequence end, window start), online softmax ----
            const bool need_mask = k0 + TILE_N > n_edge || (p.window > 0 && k0 < n_full + p.T - 1 - p.window);
            float alpha[NT][2];
            bool any_alpha = false;
            uint32_t pb[NT][4][2];     // P^T (fp16) as the second operand of O^T += V^T P^T: [16-key group][keys 0-7 / 8-15]
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int lo = (need_mask && p.window > 0) ? n_full + ((8 * nt + 2 * tq + e) % p.T) - p.window : -1;
                    float mx = -INFINITY;
#pragma unroll
                    for (int mt = 0; mt < 4; ++mt)
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
                            float v = s[nt][mt][2 * hh + e] * sscale;
                            if (need_mask) {
                                const int jj = k0 + mt * 16 + hh * 8 + g;
                                v = (jj < vis[nt][e] && jj >= lo) ? v : -INFINITY;
                            }
                            s[nt][mt][2 * hh + e] = v;
                            mx = fmaxf(mx, v);
                        }
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
                    const float mn = fmaxf(m[nt][e], mx);
                    const float ms = mn == -INFINITY ? 0.f : mn;
                    alpha[nt][e] = ex2_fast(m[nt][e] - ms);
                    any_alpha |= alpha[nt][e] != 1.f;
                    m[nt][e] = mn;
                    float sum = 0.f;
#pragma unroll
                    for (int mt = 0; mt < 4; ++mt)
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
                            const float pv = ex2_fast(s[nt][mt][2 * hh + e] - ms);
                            s[nt][mt][2 * hh + e] = pv;
                            sum += pv;
                        }
                    l[nt][e] = l[nt][e] * alpha[nt][e] + sum;
                }
                // (key g, rows 2 tq, 2 tq + 1) -> (row g, keys 2 tq, 2 tq + 1), for the first and the second
                // eight keys of every 16-key group
#pragma unroll
                for (int mt = 0; mt < 4; ++mt) {
                    pb[nt][mt][0] = movmatrix_trans(pack_f16x2(s[nt][mt][0], s[nt][mt][1]));
                    pb[nt][mt][1] = movmatrix_trans(pack_f16x2(s[nt][mt][2], s[nt][mt][3]));
                }
            }
            if (__any_sync(0xffffffffu, any_alpha)) {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int j = 0; j < 4; ++j)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            acc[nt][j][e][0] *= alpha[nt][0]; acc[nt][j][e][1] *= alpha[nt][1];
                            acc[nt][j][e][2] *= alpha[nt][0]; acc[nt][j][e][3] *= alpha[nt][1];
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
            // ---- O^T += V^T P^T.  The transposed ldmatrix hands this lane, for keys 2 tq and 2 tq + 1 of
            //      an 8-key group, the two channels 2 g and 2 g + 1 of a 16-byte chunk: the even channels of
            //      a pair of chunks form one product tile (slots 0-7 from the first chunk, 8-15 from the
            //      second), the odd ones another ----
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
                    const uint32_t e0 = e4m3x2_to_f16x2(r0), e1 = e4m3x2_to_f16x2(r2);          // even channels
                    const uint32_t e2 = e4m3x2_to_f16x2(r1), e3 = e4m3x2_to_f16x2(r3);
                    const uint32_t o0 = e4m3x2_to_f16x2(r0 >> 16), o1 = e4m3x2_to_f16x2(r2 >> 16);   // odd channels
                    const uint32_t o2 = e4m3x2_to_f16x2(r1 >> 16), o3 = e4m3x2_to_f16x2(r3 >> 16);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        mma_f16_16816(acc[nt][j][0], e0, e1, e2, e3, pb[nt][kg][0], pb[nt][kg][1]);
                        mma_f16_16816(acc[nt][j][1], o0, o1, o2, o3, pb[nt][kg][0], pb[nt][kg][1]);
                    }
                }
            }
            if (k0 + TILE_N > seg.n_kv) fence_proxy_async_smem();   // generic writes before TMA reuse
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty_bar[stage]);
        }

        // ---- merge the four warps' states, write the final rows or this segment's partial ----
        {
            float* mo = merge_o + (warp * ROWS) * D;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    l[nt][e] += __shfl_xor_sync(0xffffffffu, l[nt][e], 4);
                    l[nt][e] += __shfl_xor_sync(0xffffffffu, l[nt][e], 8);
                    l[nt][e] += __shfl_xor_sync(0xffffffffu, l[nt][e], 16);
                    const int row = 8 * nt + 2 * tq + e;
                    // the even and the odd tile of a chunk pair hold neighbouring channels
#pragma unroll
                    for (int j = 0; j < 4; ++j)
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh)
                            *reinterpret_cast<float2*>(mo + row * D + 32 * j + 16 * hh + 2 * g) =
                                make_float2(acc[nt][j][0][2 * hh + e], acc[nt][j][1][2 * hh + e]);
                    if (g == 0) {
                        merge_ml[(warp * ROWS + row) * 2] = m[nt][e];
                        merge_ml[(warp * ROWS + row) * 2 + 1] = l[nt][e];
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
            const float outv = L > 0.f ? acc / L * vscale : 0.f;
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
