// Launch interfaces of the kernels (device code lives in the *_kernel.cu files).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cstdint>

#include "plan.h"

namespace yoco {

constexpr int32_t kStatusOk = 0;
// Status word (first int32 of a workspace, or the append kernel's own word): 0 = ok, otherwise
//   bits 0-7   which kind of wait ran out (WaitClass)
//   bits 8-31  1 + linear index of the CTA that gave up first
// The first failure wins (compare-and-swap against 0), so the word names where the trouble began.
enum WaitClass : int32_t {
    kWaitItemQueue = 1,   // decode: next work item from the producer / queue entry read by the consumers
    kWaitRingFull = 2,    // a consumer waiting for a K/V (or Q, X, W) tile to land
    kWaitRingEmpty = 3,   // the producer waiting for a stage to be released
    kWaitTensor = 4,      // a tensor-core hand-over: scores ready, P written, product finished
    kWaitDrain = 5,       // leaving: a copy or product that had been started did not finish in time
    kWaitMisaligned = 6,  // dynamic shared memory not 1 KB aligned (no wait involved; nothing ran)
};
__host__ __device__ constexpr int32_t status_word(int32_t wait_class, int32_t cta) {
    return wait_class | ((cta + 1) << 8);
}


// Work tables small enough to travel as kernel parameters (the decode call then needs no
// host-to-device copy): every benchmark shape fits; larger problems read them from the workspace.
constexpr int kInlineSegments = 448;
constexpr int kInlineGroups = 303;
constexpr int kInlineStreams = 256;
struct DecodeInlineTables {
    DevSegment seg[kInlineSegments];
    int32_t group_begin[kInlineGroups + 1];
};
struct CombineInlineTables {
    int32_t stream_base[kInlineStreams];
    int32_t stream_nseg[kInlineStreams];
};

struct CombineParams {
    int64_t rows;               // output rows (B*Hq*T, or the public `rows`)
    int32_t d;
    // public layout ([rows][S][d]) when stream_base == nullptr
    int32_t S;
    // internal slot-major layout
    int32_t Hq, Hkv, T, rows_per_stream;
    int32_t max_pieces;         // most pieces any row has (S, or the plan's max_splits): picks the launch shape
    int32_t sub_items;          // internal layout: slots per table entry (0 or 1: one)
    const int32_t* stream_base; // [B*Hkv] first slot of each stream
    const int32_t* stream_nseg; // [B*Hkv] slots of each stream
    const float* part_o;
    const float* part_lse;      // natural log, -inf = empty
    __nv_bfloat16* O;           // [rows, d] bf16 result, or null when O_f32 is given
    float* lse;                 // may be null
    float* O_f32;               // [rows, d] fp32 result instead of O (a partial result that another
                                // merge will consume: key-range sharding across GPUs)
    int32_t merge_unsplit;      // internal layout: also copy rows whose stream has a single piece
                                // (set when the attention kernel was told to write no final rows)
    int32_t piece_major;        // public layout is [S][rows][d] / [S][rows] (as an all-gather over S
                                // ranks leaves it) instead of [rows][S][d] / [rows][S]
};
// inline_tab (host, may be null): stream tables passed as kernel parameters instead of
// p.stream_base / p.stream_nseg.  after_attention: launched right behind the attention kernel of
// the same call; the launch is then allowed to overlap that kernel's tail (the merge itself still
// waits for it).
cudaError_t launch_combine(const CombineParams& p, cudaStream_t stream,
                           const CombineInlineTables* inline_tab = nullptr, bool after_attention = false);

struct DecodeParams {
    const __nv_bfloat16* Q;     // [B*Hq*T, d]
    __nv_bfloat16* O;           // [B*Hq*T, d]
    float* lse;                 // [B*Hq*T] or null
    const DevSegment* segments;
    const int32_t* group_begin; // [num_groups + 1]
    float* part_o;              // [num_segments][rows_per_stream][d]
    float* part_lse;            // [num_segments][rows_per_stream]
    int32_t* status;
    float scale_log2;           // scale * log2(e)
    int32_t T;
    int32_t rows_per_stream;    // G * T (<= 16)
    int32_t d;
    int32_t window;             // sliding window C, 0 = none
    int32_t force_partial;      // write every segment to its partial slot, even of an unsplit stream
    int32_t sub_items;          // pieces per group (plan.h: sub_bound); slot = segment slot * sub_items + piece
    int32_t* work_counter;      // zeroed before the launch; hands out the pieces beyond each CTA's first
    int64_t wait_limit_ns;      // 0 = the default limit of a bounded wait
    int32_t selftest_skip_loads;// self-test of the give-up path: the producer arms no copy, so the first
                                // consumer wait runs out (with nothing in flight) and the kernel returns
};
// tmK / tmV: 2-D tensor maps over the [rows, d] view of K and V, box {64, kDecodeTileN},
// 128-byte swizzle.
// inline_tab (host, may be null): segments and group offsets passed as kernel parameters instead
// of p.segments / p.group_begin.
cudaError_t launch_decode(const DecodeParams& p, const CUtensorMap& tmK, const CUtensorMap& tmV,
                          int num_groups, cudaStream_t stream, const DecodeInlineTables* inline_tab = nullptr);
// one-time per-device kernel attribute set-up (dynamic shared memory opt-in)
cudaError_t decode_kernel_setup();


// ---- decode over an 8-bit (FP8 E4M3) cache, head dimension 128 ---------------------------------
constexpr int kFp8MaxHeads = 64;
struct DecodeFp8Params {
    DecodeParams base;                    // as for the bf16 kernel; base.scale_log2 is unused
    int32_t Hkv;
    float score_scale_log2[kFp8MaxHeads]; // per KV head: softmax scale * k_scale[c] * log2(e)
    float v_scale[kFp8MaxHeads];          // per KV head
};
// tmK / tmV: 2-D uint8 tensor maps over the [rows, 128] byte view of K and V, box {128, 64},
// 128-byte swizzle.
cudaError_t launch_decode_fp8(const DecodeFp8Params& p, const CUtensorMap& tmK, const CUtensorMap& tmV,
                              int num_groups, cudaStream_t stream, const DecodeInlineTables* inline_tab);
cudaError_t decode_fp8_kernel_setup();

struct ChunkParams {
    __nv_bfloat16* O;           // [B*Hq*T, d]
    float* lse;                 // [B*Hq*T] or null
    const DevSegment* segments;
    const int32_t* group_begin; // [num_groups + 1]
    float* part_o;              // [num_segments][rows_per_stream][d]
    float* part_lse;            // [num_segments][rows_per_stream]
    int32_t* status;
    float scale_log2;           // scale * log2(e)
    int32_t T;
    int32_t rows_per_stream;    // G * T
    int32_t m_tiles;            // ceil(rows_per_stream / 128)
    int32_t d;
    int32_t window;             // sliding window C, 0 = none
    int32_t force_partial;      // write every segment to its partial slot, even of an unsplit stream
};
// tmQ: [B*Hq*T, d] box {64, 128}; tmK / tmV: [rows, d] box {64, kChunkTileN}; 128-byte swizzle.
// Grid = num_groups * m_tiles CTAs, the row tile varying fastest so that the CTAs that walk the
// same K/V range run side by side and share it through L2.
cudaError_t launch_chunk(const ChunkParams& p, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                         const CUtensorMap& tmV, int num_groups, cudaStream_t stream);
cudaError_t chunk_kernel_setup();
// Same interface for streams with more than 128 rows: one CTA owns two 128-row tiles (m_tiles =
// ceil(rows_per_stream / 256)), tmQ box is still {64, 128}.
// fp8_scales (host, may be null): K and V are an 8-bit cache (tmK / tmV then are uint8 maps over the
// [rows, 128] byte view, box {128, kChunkTileN}); head dimension 128 only.
struct ChunkFp8Scales {
    int32_t Hkv;
    float score_scale_log2[kFp8MaxHeads]; // per KV head: softmax scale * k_scale[c] * log2(e)
    float v_scale[kFp8MaxHeads];          // per KV head
};
cudaError_t launch_chunk_pair(const ChunkParams& p, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                              const CUtensorMap& tmV, int num_groups, cudaStream_t stream,
                              const ChunkFp8Scales* fp8_scales = nullptr);
cudaError_t chunk_pair_kernel_setup();

// ---- writing the cache: K^ = RMSNorm(X) W_K, V^ = RMSNorm(X) W_V appended head-major ------------
constexpr int kAppendMaxSequences = 512;
struct KvAppendParams {
    const __nv_bfloat16* X;     // [M, d_model] (the few-token kernel reads it with plain loads)
    __nv_bfloat16* K;           // packed head-major caches
    __nv_bfloat16* V;
    int32_t M;                  // B * T tokens
    int32_t T, d, d_model;
    int32_t n_half;             // Hkv * d: output columns of K^ (those of V^ follow)
    float eps;
};
struct KvAppendTables {         // per sequence, as kernel parameters
    int32_t row0[kAppendMaxSequences];       // cache row (units of d elements) of (head 0, key N_i - T)
    int32_t head_rows[kAppendMaxSequences];  // rows between two heads of the sequence
};
// tmX: [M, d_model] box {64, 128}; tmWk / tmWv: gain-folded weights [d_model, Hkv*d] box {64, 128};
// 128-byte swizzle.  Grid = (2*Hkv*d/128, ceil(M/128)); with M <= 16 tokens (a decode step) a second
// kernel streams the weights instead: clusters of CTAs split d_model and add up through
// distributed shared memory.
struct KvAppendScales {         // 8-bit cache: reciprocal of the per-head scales (value = scale * e4m3(byte))
    float inv_k[kFp8MaxHeads];
    float inv_v[kFp8MaxHeads];
};
// fp8_scales (host, may be null): store FP8 E4M3 bytes instead of bf16.
cudaError_t launch_kv_append(const KvAppendParams& p, const KvAppendTables& tab, const CUtensorMap& tmX,
                             const CUtensorMap& tmWk, const CUtensorMap& tmWv, cudaStream_t stream,
                             const KvAppendScales* fp8_scales = nullptr);
cudaError_t launch_fold_gain(const __nv_bfloat16* g, const __nv_bfloat16* W, __nv_bfloat16* Wg, int64_t d_model,
                             int64_t n_out, cudaStream_t stream);
cudaError_t read_and_clear_kv_append_status(int32_t* word, cudaStream_t stream);
cudaError_t kv_append_kernel_setup();

}  // namespace yoco
