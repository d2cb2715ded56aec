// Log-sum-exp merge of partial attention results (the second kernel of the split-KV path).
//
//   lse = log sum_s exp(lse_s),   O = sum_s exp(lse_s - lse) * O_s
//
// One warp per output row; lanes cover the head dimension with 128-bit loads.
#include "kernels.h"

namespace yoco {

namespace {

constexpr int kCombineWarps = 4;

// VEC = floats per lane (d = 32 * VEC for the packed widths, else generic loop)
__global__ void __launch_bounds__(kCombineWarps * 32)
combine_kernel(CombineParams p) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * kCombineWarps + warp;
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
        const int slot0 = p.stream_base[stream];
        nseg = p.stream_nseg[stream];
        if (nseg == 1) return;   // an unsplit stream: the attention kernel wrote the final rows itself
        o_base = ((int64_t)slot0 * p.rows_per_stream + r_local) * p.d;
        o_stride = (int64_t)p.rows_per_stream * p.d;
        lse_base = (int64_t)slot0 * p.rows_per_stream + r_local;
        lse_stride = p.rows_per_stream;
    } else {
        // public layout: [rows][S][d]
        nseg = p.S;
        o_base = row * p.S * p.d;
        o_stride = p.d;
        lse_base = row * p.S;
        lse_stride = 1;
    }

    float m = -INFINITY;
    for (int s = lane; s < nseg; s += 32) m = fmaxf(m, p.part_lse[lse_base + s * lse_stride]);
#pragma unroll
    for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));

    __nv_bfloat16* out = p.O + row * p.d;
    if (m == -INFINITY) {   // no piece carries weight (also nseg == 0)
        for (int e = lane; e < p.d; e += 32) out[e] = __float2bfloat16(0.f);
        if (p.lse && lane == 0) p.lse[row] = -INFINITY;
        return;
    }
    float denom = 0.f;
    for (int s = lane; s < nseg; s += 32) {
        const float l = p.part_lse[lse_base + s * lse_stride];
        if (l != -INFINITY) denom += __expf(l - m);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) denom += __shfl_xor_sync(0xffffffffu, denom, o);
    const float inv = 1.f / denom;

    // each lane owns 4 consecutive channels per 128-channel block
    for (int e0 = lane * 4; e0 < p.d; e0 += 128) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s = 0; s < nseg; ++s) {
            const float l = p.part_lse[lse_base + s * lse_stride];
            if (l == -INFINITY) continue;
            const float w = __expf(l - m) * inv;
            const float4 v = *reinterpret_cast<const float4*>(p.part_o + o_base + s * o_stride + e0);
            acc.x += w * v.x; acc.y += w * v.y; acc.z += w * v.z; acc.w += w * v.w;
        }
        __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
        uint2 pk;
        pk.x = *reinterpret_cast<uint32_t*>(&lo);
        pk.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(out + e0) = pk;
    }
    if (p.lse && lane == 0) p.lse[row] = m + __logf(denom);
}

}  // namespace

cudaError_t launch_combine(const CombineParams& p, cudaStream_t stream) {
    if (p.rows == 0) return cudaSuccess;
    const int64_t blocks = (p.rows + kCombineWarps - 1) / kCombineWarps;
    combine_kernel<<<(unsigned)blocks, kCombineWarps * 32, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace yoco
