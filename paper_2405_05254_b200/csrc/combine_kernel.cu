// Log-sum-exp merge of partial attention results (the second kernel of the split-KV path).
//
//   lse = log sum_s exp(lse_s),   O = sum_s exp(lse_s - lse) * O_s
//
// Lanes cover the head dimension with 128-bit loads.  With few pieces per row one warp merges a
// row; with many (a long sequence cut into dozens or hundreds of pieces) the 4 or 32 warps of a
// CTA share the pieces of one row, and the loop carries no load-to-branch dependence, so that
// several pieces are in flight at once: the merge is a chain of dependent memory latencies
// otherwise, and its length is what the launch shape is chosen to bound.
#include "kernels.h"

namespace yoco {

namespace {

constexpr int kCombineWarps = 4;       // warps per CTA of the small shapes
constexpr int kCombineWarpsMany = 32;  // one 1024-thread CTA per row when a row has very many pieces
constexpr int kManyPieces = 64;

// WPR: warps per output row (1 or WARPS); WARPS: warps per CTA
template <int WPR, int WARPS>
__device__ __forceinline__ void combine_body(const CombineParams& p) {
    // When launched behind the attention kernel with programmatic stream serialisation, this
    // grid may start before that kernel has finished: wait for it (and for its writes) here.
    // Without that launch attribute the instruction returns at once.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t row = WPR == 1 ? (int64_t)blockIdx.x * WARPS + warp : (int64_t)blockIdx.x;
    const int sub = WPR == 1 ? 0 : warp;
    if (row >= p.rows) return;

    // where this row's partials live
    int64_t o_base, lse_base, o_stride, lse_stride;
    int nseg;
    if (p.stream_base) {
        // internal layout: slot-major [slot][rows_per_stream][d]; row = (b, h, t)
        const int64_t bh = row / p.T;
        const int t = (int)(row - bh * p.T);
        const int b = (int)(bh / p.Hq), h = (int)(bh - (int64_t)b * p.Hq);
        const int G = p.Hq / p.Hkv;
        const int stream = b * p.Hkv + h / G;
        const int r_local = (h % G) * p.T + t;
        // every table entry stands for sub_items consecutive slots (the pieces of one segment)
        const int per = p.sub_items > 1 ? p.sub_items : 1;
        const int slot0 = p.stream_base[stream] * per;
        nseg = p.stream_nseg[stream] * per;
        // an unsplit stream: the attention kernel wrote the final rows itself (unless told not to)
        if (nseg == 1 && !p.merge_unsplit) return;
        o_base = ((int64_t)slot0 * p.rows_per_stream + r_local) * p.d;
        o_stride = (int64_t)p.rows_per_stream * p.d;
        lse_base = (int64_t)slot0 * p.rows_per_stream + r_local;
        lse_stride = p.rows_per_stream;
    } else {
        nseg = p.S;
        if (p.piece_major) {     // [S][rows][d]
            o_base = row * p.d;
            o_stride = p.rows * p.d;
            lse_base = row;
            lse_stride = p.rows;
        } else {                 // [rows][S][d]
            o_base = row * p.S * p.d;
            o_stride = p.d;
            lse_base = row * p.S;
            lse_stride = 1;
        }
    }

    // The partial rows this warp will need do not depend on the weights: ask for the first U of them
    // now, so that they travel while the log-sum-exps are read and reduced (one memory round trip
    // instead of two or more; U covers all of a warp's pieces in the launch shapes used).
    constexpr int U = WPR == 1 ? 4 : (WARPS == kCombineWarpsMany ? 2 : 10);
    const int e0 = lane * 4;
    float4 pre[U][2];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int s = sub + u * WPR;
#pragma unroll
        for (int blk = 0; blk < 2; ++blk)
            if (s < nseg && e0 + blk * 128 < p.d)
                pre[u][blk] = *reinterpret_cast<const float4*>(p.part_o + o_base + s * o_stride + e0 + blk * 128);
    }

    float m = -INFINITY;
    for (int s = lane; s < nseg; s += 32) m = fmaxf(m, p.part_lse[lse_base + s * lse_stride]);
#pragma unroll
    for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));

    __nv_bfloat16* out = p.O ? p.O + row * p.d : nullptr;
    float* out32 = p.O_f32 ? p.O_f32 + row * p.d : nullptr;
    if (m == -INFINITY) {   // no piece carries weight (also nseg == 0); the same for every warp of the row
        if (sub == 0) {
            for (int e = lane; e < p.d; e += 32) {
                if (out32) out32[e] = 0.f;
                else out[e] = __float2bfloat16(0.f);
            }
            if (p.lse && lane == 0) p.lse[row] = -INFINITY;
        }
        return;
    }
    float denom = 0.f;
    for (int s = lane; s < nseg; s += 32) {
        const float l = p.part_lse[lse_base + s * lse_stride];
        denom += l == -INFINITY ? 0.f : __expf(l - m);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) denom += __shfl_xor_sync(0xffffffffu, denom, o);
    const float inv = 1.f / denom;

    // each lane owns 4 consecutive channels of each 128-channel block (d <= 256: two blocks)
    float4 acc[2] = {make_float4(0.f, 0.f, 0.f, 0.f), make_float4(0.f, 0.f, 0.f, 0.f)};
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int s = sub + u * WPR;
        if (s < nseg) {
            const float l = p.part_lse[lse_base + s * lse_stride];
            const float w = l == -INFINITY ? 0.f : __expf(l - m) * inv;
#pragma unroll
            for (int blk = 0; blk < 2; ++blk) {
                if (e0 + blk * 128 < p.d) {
                    const float4 v = pre[u][blk];
                    // an empty piece may hold anything: select, never multiply by zero
                    acc[blk].x += w != 0.f ? w * v.x : 0.f;
                    acc[blk].y += w != 0.f ? w * v.y : 0.f;
                    acc[blk].z += w != 0.f ? w * v.z : 0.f;
                    acc[blk].w += w != 0.f ? w * v.w : 0.f;
                }
            }
        }
    }
#pragma unroll 4
    for (int s = sub + U * WPR; s < nseg; s += WPR) {
        const float l = p.part_lse[lse_base + s * lse_stride];
        const float w = l == -INFINITY ? 0.f : __expf(l - m) * inv;
        const float* src = p.part_o + o_base + s * o_stride;
#pragma unroll
        for (int blk = 0; blk < 2; ++blk) {
            if (e0 + blk * 128 < p.d) {
                const float4 v = *reinterpret_cast<const float4*>(src + e0 + blk * 128);
                // an empty piece may hold anything: select, never multiply by zero
                acc[blk].x += w != 0.f ? w * v.x : 0.f;
                acc[blk].y += w != 0.f ? w * v.y : 0.f;
                acc[blk].z += w != 0.f ? w * v.z : 0.f;
                acc[blk].w += w != 0.f ? w * v.w : 0.f;
            }
        }
    }
    if (WPR > 1) {
        __shared__ float4 red[WARPS][2][32];
        red[warp][0][lane] = acc[0];
        red[warp][1][lane] = acc[1];
        __syncthreads();
        if (warp != 0) return;
#pragma unroll
        for (int blk = 0; blk < 2; ++blk) {
            float4 t = red[0][blk][lane];
#pragma unroll
            for (int w2 = 1; w2 < WARPS; ++w2) {
                const float4 u = red[w2][blk][lane];
                t.x += u.x; t.y += u.y; t.z += u.z; t.w += u.w;
            }
            acc[blk] = t;
        }
    }
#pragma unroll
    for (int blk = 0; blk < 2; ++blk) {
        if (e0 + blk * 128 < p.d && out32) {
            *reinterpret_cast<float4*>(out32 + e0 + blk * 128) = acc[blk];
        } else if (e0 + blk * 128 < p.d) {
            __nv_bfloat162 lo = __floats2bfloat162_rn(acc[blk].x, acc[blk].y), hi = __floats2bfloat162_rn(acc[blk].z, acc[blk].w);
            uint2 pk;
            pk.x = *reinterpret_cast<uint32_t*>(&lo);
            pk.y = *reinterpret_cast<uint32_t*>(&hi);
            *reinterpret_cast<uint2*>(out + e0 + blk * 128) = pk;
        }
    }
    if (p.lse && lane == 0) p.lse[row] = m + __logf(denom);
}

template <int WPR, int WARPS>
__global__ void __launch_bounds__(WARPS * 32) combine_kernel(const CombineParams p) { combine_body<WPR, WARPS>(p); }

// stream tables as kernel parameters
template <int WPR, int WARPS>
__global__ void __launch_bounds__(WARPS * 32)
combine_kernel_inline(const CombineParams p0, const __grid_constant__ CombineInlineTables tab) {
    CombineParams p = p0;
    p.stream_base = tab.stream_base;
    p.stream_nseg = tab.stream_nseg;
    combine_body<WPR, WARPS>(p);
}

}  // namespace

cudaError_t launch_combine(const CombineParams& p, cudaStream_t stream, const CombineInlineTables* inline_tab,
                           bool after_attention) {
    if (p.rows == 0) return cudaSuccess;
    // pieces per row -> shape: a warp per row; a 4-warp CTA per row; a 32-warp CTA per row
    const int shape = p.max_pieces > kManyPieces ? 2 : p.max_pieces > kCombineWarps ? 1 : 0;
    const int warps = shape == 2 ? kCombineWarpsMany : kCombineWarps;
    const int64_t blocks = shape ? p.rows : (p.rows + kCombineWarps - 1) / kCombineWarps;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(warps * 32);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = after_attention ? 1 : 0;
    if (inline_tab) {
        if (shape == 2)
            return cudaLaunchKernelEx(&cfg, combine_kernel_inline<kCombineWarpsMany, kCombineWarpsMany>, p, *inline_tab);
        if (shape == 1) return cudaLaunchKernelEx(&cfg, combine_kernel_inline<kCombineWarps, kCombineWarps>, p, *inline_tab);
        return cudaLaunchKernelEx(&cfg, combine_kernel_inline<1, kCombineWarps>, p, *inline_tab);
    }
    if (shape == 2) return cudaLaunchKernelEx(&cfg, combine_kernel<kCombineWarpsMany, kCombineWarpsMany>, p);
    if (shape == 1) return cudaLaunchKernelEx(&cfg, combine_kernel<kCombineWarps, kCombineWarps>, p);
    return cudaLaunchKernelEx(&cfg, combine_kernel<1, kCombineWarps>, p);
}

}  // namespace yoco
