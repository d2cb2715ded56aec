/*
 * yoco_xattn -- cross-decoder attention over the single shared K/V cache of the
 * decoder-decoder architecture (Section 2.2, the cross-decoder equation block:
 * Q^l = LN(X^l) W_Q^l,  Y^l = Attention(Q^l, K^, V^) + X^l, "standard multi-head
 * attention", causal, grouped-query).  This library computes the Attention(...)
 * term only:  O = softmax(scale * Q K^T + causal mask) V  per sequence and head.
 *
 * Every cross-decoder layer calls it with its own Q and the SAME K/V pointers
 * (the cache is written once by the self-decoder and reused by all L/2 layers).
 *
 * C ABI, sm_100a only.  No call allocates or frees device memory, none
 * synchronises the host with the device unless stated, none throws.
 *
 * ---------------------------------------------------------------------------
 * Layouts (all tensors contiguous, bf16 = 16-bit bfloat bit patterns)
 *
 *   Q, O   [B, Hq, T, d]   device.  Query head h reads KV head h / G, G = Hq / Hkv.
 *   K, V   packed device buffers.  Sequence i starts at TOKEN offset cu_kv[i];
 *          inside a sequence the order is head-major [Hkv, N_i, d]:
 *            element(i, c, j, e) = cu_kv[i]*Hkv*d + c*head_stride_i + j*d + e
 *          head_stride_i = kv_head_stride if non-zero (a cache with spare
 *          capacity per head; must be a multiple of d), else N_i*d (tight).
 *          With equal lengths and tight packing this is [B, Hkv, N, d].
 *          A sequence occupies Hkv * head_stride_i elements from its offset, so
 *          cu_kv[i+1] - cu_kv[i] >= head_stride_i / d is required (else INVALID_ARG).
 *          Both buffers must start on a 16-byte boundary.
 *   kv_len[i] = N_i  counts ALL keys of sequence i including the T positions of
 *          the current call (the self-decoder has already appended them).
 *   Causal rule: query row t (0-based, T rows) sits at position i = N_i - T + t and sees keys
 *          j <= i.  T = 1 sees the whole cache.  With shape.window = C > 0 it sees only
 *          i - C < j <= i (the sliding-window mask of Section 3.2, B_ij = 0 iff i - C < j <= i);
 *          keys that no row of the call can see are neither read nor planned.  A row with no visible key yields O = 0
 *          and LSE = -inf.
 *   LSE    [B, Hq, T] fp32, natural logarithm of sum_j exp(scale * q.k_j); optional.
 *
 * Ownership: every pointer is caller-owned and must stay valid until the
 * stream has executed the call.  `stream` is a cudaStream_t passed as void*
 * (NULL = legacy default stream).  Work is only enqueued; calls return
 * immediately.  The workspace may be reused by the next call on the same
 * stream; calls on different streams need different workspaces.
 *
 * Errors: every function returns YOCO_OK or a negative code.  Argument and
 * shape checks happen before anything is enqueued.  A device-side bounded wait
 * that ran out (never expected) is recorded in a status word inside the
 * workspace and read back by yoco_xattn_status(); the kernel that gave up first
 * waits for the copies and products it had started, then returns normally, so the
 * context stays usable.
 *
 * CUDA graphs: a call may be recorded into a graph.  The work tables of a problem
 * with at most 448 work segments, 303 CTA groups and 256 (sequence, KV head) streams
 * travel as kernel parameters and the recorded nodes refer to nothing but the
 * caller's buffers.  A larger problem uploads its tables from host memory owned by
 * the library's plan cache; the library then keeps that plan for the life of the
 * process, so a replay never reads released memory.  In both cases the caller's
 * buffers, kv_len and cu_kv as they were at recording time are what a replay uses.
 */
#ifndef YOCO_XATTN_H_
#define YOCO_XATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define YOCO_OK                        0
#define YOCO_ERR_INVALID_ARG          (-1)  /* null pointer, negative size, misaligned buffer   */
#define YOCO_ERR_UNSUPPORTED          (-2)  /* d not in {64,128}, Hq % Hkv != 0, G*T too large  */
#define YOCO_ERR_WORKSPACE_TOO_SMALL  (-3)
#define YOCO_ERR_CUDA                 (-4)  /* a CUDA call failed; see yoco_xattn_last_cuda_error */
#define YOCO_ERR_TIMEOUT              (-5)  /* a bounded device-side wait expired               */
#define YOCO_ERR_STATIC_SCRATCH_EXCEEDED (-6) /* yoco_xattn_decode_static: problem too large    */

#define YOCO_MODE_DECODE 0   /* split-KV kernel, G*T <= 16 query rows per KV head        */
#define YOCO_MODE_CHUNK  1   /* tensor-core (tcgen05) kernel, any T >= 1                 */

typedef struct yoco_xattn_shape {
    int32_t B;               /* sequences                                                 */
    int32_t Hq;              /* query heads                                               */
    int32_t Hkv;             /* key/value heads, divides Hq                               */
    int32_t d;               /* head dimension: 64 or 128                                 */
    int32_t T;               /* query rows per sequence in this call                      */
    float   scale;           /* > 0, or 0 -> 1/sqrt(d); negative values are rejected       */
    int64_t kv_head_stride;  /* elements between KV heads of one sequence; 0 -> N_i*d     */
    int32_t max_kv_len;      /* used as every N_i when kv_len_host is NULL                */
    int32_t window;          /* sliding window C (Section 3.2: row i sees i - C < j <= i);
                                0 = none (plain causal); negative values are rejected     */
} yoco_xattn_shape;

/* One unit of work: a contiguous key range of one (sequence, KV head) stream,
 * executed by CTA group `group`; its partial result goes to slot `slot`. */
typedef struct yoco_xattn_segment {
    int32_t group;      /* work item: CTA group g, or with sub_items > 1 piece r of
                           group g as r * num_groups + g                                  */
    int32_t b;          /* sequence                                                       */
    int32_t c;          /* KV head                                                        */
    int32_t k_begin;    /* first key (multiple of tile_n)                                 */
    int32_t k_end;      /* one past the last key (multiple of tile_n, or N_i)             */
    int32_t slot;       /* partial-result slot; slots of one stream are consecutive       */
} yoco_xattn_segment;

typedef struct yoco_xattn_plan_info {
    int32_t mode;            /* YOCO_MODE_*                                               */
    int32_t tile_n;          /* keys per shared-memory tile                               */
    int32_t tile_m;          /* query rows per CTA: 16 decode; chunk 128, or 256 (two
                                tensor-core tiles sharing K/V) when G*T > 128             */
    int32_t m_tiles;         /* row tiles per stream = ceil(G*T / tile_m)                 */
    int32_t num_groups;      /* CTA groups; each streams one contiguous range of the flat
                                (stream, key tile) space                                  */
    int32_t num_ctas;        /* grid size = num_groups * m_tiles                          */
    int32_t num_streams;     /* B * Hkv                                                   */
    int32_t num_segments;    /* total work segments = number of partial slots             */
    int32_t max_splits;      /* most segments any one stream was cut into                 */
    int32_t needs_combine;   /* 0 when every stream has exactly one segment               */
    int64_t total_tiles;     /* sum over streams of ceil(N_i / tile_n)                    */
    int64_t workspace_bytes; /* what decode/chunk need for this problem                   */
    int32_t sub_items;       /* decode: pieces a group's range is cut into (1, 2 or 4)    */
    int32_t num_slots;       /* partial-result slots the workspace holds                  */
} yoco_xattn_plan_info;

/* Split-count / tile heuristic (host only, integers only, deterministic).  No counterpart in the
 * paper, which names no kernel for cross-attention (Section 4.4 attributes split-KV decoding only
 * to its Transformer baseline); exported so that tests can check the plan integer for integer.
 * The flat space of (stream, key tile) pairs, streams ordered (b, c), is cut into
 * num_groups contiguous ranges of equal tile count (+-1); a range that crosses a
 * stream boundary becomes several segments.  num_groups = min(total_tiles,
 * sm_count * groups_per_sm(mode)).  sm_count > 0 must be given (pure host call).
 * Decode plans whose groups are long (>= 40 tiles) and made of long runs (at most two segments
 * per group on average) cut every group's range once more, into
 * sub_items pieces of decreasing size (yoco_xattn_sub_bound): the SMs of a GPU do not all
 * stream at the same rate, so CTA g runs piece 0 of its own group and the remaining pieces
 * are handed out, in item order, to whichever CTA is free.  The pieces, their slots and the
 * merge order are fixed here, so the result is the same whoever runs a piece; segments_out
 * then lists the pieces.  (yoco_xattn_decode_static runs with sub_items = 1;
 * yoco_xattn_decode_fp8 chooses the pieces as for half as many tiles, a tile of an 8-bit cache
 * being half the bytes.)
 * kv_len_host: [B] or NULL (every N_i = shape->max_kv_len).
 * segments_out: optional array of `capacity` entries; at most `capacity` are written,
 * info->num_segments tells how many exist.  */
int32_t yoco_xattn_plan(const yoco_xattn_shape* shape, const int32_t* kv_len_host,
                        int32_t sm_count, int32_t mode, yoco_xattn_plan_info* info,
                        yoco_xattn_segment* segments_out, int32_t capacity);

/* (No counterpart in the paper.)  First tile, counted inside a group of n_tiles key tiles, of piece r of sub_items
 * (r = 0 .. sub_items; sub_items in {1, 2, 4}): piece r covers tiles [bound(r), bound(r+1))
 * with bound(r) = n_tiles * c(r) / 64 rounded down, c = 0, 52, 64 for two pieces and
 * 0, 44, 54, 61, 64 for four.  Returns -1 for other arguments.  Pure host. */
int64_t yoco_xattn_sub_bound(int64_t n_tiles, int32_t sub_items, int32_t r);

/* (No counterpart in the paper.)  Workspace bytes for decode/chunk on this problem.  sm_count = 0 queries the
 * current CUDA device (then YOCO_ERR_CUDA is possible).  Pure host otherwise. */
int32_t yoco_xattn_workspace_size(const yoco_xattn_shape* shape, const int32_t* kv_len_host,
                                  int32_t sm_count, int32_t mode, size_t* bytes);

/* Attention(Q^l, K^, V^) of Section 2.2 (cross-decoder equations) for the next-token call of a
 * cross-decoder layer, the call whose cost Section 2.3 reduces to one pass over the single shared
 * cache: split-KV decode (flash-decoding style) of a few query rows per KV head (G*T <= 16;
 * typically T = 1) against the whole cache.  Runs the split kernel, then the merge when a stream was split.
 *   Q, K, V, O, lse (may be NULL), workspace: device.  cu_kv_host: host [B+1] token
 *   offsets, or NULL = prefix sums of kv_len (tight packing).  kv_len_host: host [B]
 *   or NULL.  workspace: >= yoco_xattn_workspace_size(), 256-byte aligned; it holds the
 *   status word, the work counter of the run-time piece assignment, the work tables and the
 *   partial results of THIS call: successive calls on one stream may share it (the 13 layer
 *   calls of a step do), calls that can overlap on the GPU need one each.  Its contents need
 *   no initialisation and mean nothing after the call except to yoco_xattn_status.   */
int32_t yoco_xattn_decode(const yoco_xattn_shape* shape, const void* Q, const void* K,
                          const void* V, const int32_t* cu_kv_host, const int32_t* kv_len_host,
                          void* O, float* lse, void* workspace, size_t workspace_bytes,
                          void* stream);

/* Decode without a workspace argument.  (The paper has no counterpart: this is a packaging
 * variant of yoco_xattn_decode, same kernels, same result.)
 *
 * Who needs it: code that may not create device memory at the point where it calls
 * attention -- a plugin inside a host application that owns the allocator, a real-time loop
 * that forbids cudaMalloc after start-up, a caller whose memory pool is sized and frozen in
 * advance.  Such callers still pass Q, K, V, O (and lse), but the split tables and the partial
 * results go to a 4 MiB buffer that is part of this library's device image.  Every GPU that
 * loads the library carries those 4 MiB until the process ends.
 *
 * Limits and rules:
 *  - A problem whose one-piece decode plan (every CTA group a single work piece, which is how this
 *    entry always runs; at most what yoco_xattn_workspace_size reports for decode mode) needs more
 *    than yoco_xattn_static_scratch_bytes() is refused with YOCO_ERR_STATIC_SCRATCH_EXCEEDED and
 *    nothing is enqueued.  4 MiB covers, e.g., B = 1 at 1M tokens and 16 ragged sequences.
 *  - The status word of these calls lives in the built-in buffer: yoco_xattn_status(NULL, stream)
 *    reads it (for the current device).
 *  - No cudaMalloc / cudaFree and no allocating library routine is called.
 *  - The first call on each device looks the buffer's device address up (and sets kernel
 *    attributes); make that first call with the device current and before any stream capture.
 *  - All calls on a device share the one buffer, and it keeps whatever the previous call left.
 *    The library rewrites the tables and the status word at the start of every call, and every
 *    partial result is written before it is read, so stale contents are never used.  Two calls
 *    that can overlap on the GPU (different streams without an ordering between them) race on
 *    the buffer: order them, or give one of them yoco_xattn_decode with its own workspace.
 *  - Argument and size errors are returned directly, before anything is enqueued. */
int32_t yoco_xattn_decode_static(const yoco_xattn_shape* shape, const void* Q, const void* K,
                                 const void* V, const int32_t* cu_kv_host,
                                 const int32_t* kv_len_host, void* O, float* lse, void* stream);

/* (No counterpart in the paper.)  Size in bytes of the built-in buffer used by yoco_xattn_decode_static. */
int32_t yoco_xattn_static_scratch_bytes(void);

/* Attention(Q^l, K^, V^) of Section 2.2 for many positions at once ("causal masking is also used
 * for cross-attention"): a prefill or scoring chunk, whose cost is the O(N) per position of
 * Section 2.3's prefill table.  T new query rows per sequence, causal
 * inside the chunk, as a dense contraction on the tcgen05 tensor cores (S = Q K^T
 * and O = P V with accumulators in tensor memory).  Same arguments as decode; any
 * T >= 1.  */
int32_t yoco_xattn_chunk(const yoco_xattn_shape* shape, const void* Q, const void* K,
                         const void* V, const int32_t* cu_kv_host, const int32_t* kv_len_host,
                         void* O, float* lse, void* workspace, size_t workspace_bytes,
                         void* stream);

/* (No counterpart in the paper: the exact recombination of softmax attention evaluated over
 * disjoint key ranges.)  Stand-alone log-sum-exp merge of S partial attention results per row:
 *   lse = log sum_s exp(lse_s),   O = sum_s exp(lse_s - lse) * O_s
 * part_o [rows, S, d] fp32 (each O_s already normalised), part_lse [rows, S] fp32
 * natural log, -inf marks an empty piece (weight 0; all empty -> O = 0, lse = -inf).
 * O [rows, d] bf16, lse [rows] fp32 or NULL.  All device pointers.  d % 8 == 0, d <= 256.
 * Also the local step of key-range sharding across GPUs (exchange partials, merge). */
int32_t yoco_xattn_combine(int64_t rows, int32_t S, int32_t d, const float* part_o,
                           const float* part_lse, void* O, float* lse, void* stream);

/* Decode over an 8-bit cache (Section 1 assumes 8-bit K/V quantisation when it sizes a cache): K8, V8 hold FP8 E4M3
 * bytes (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities) in the packed
 * head-major layout described above, one byte per element (offsets and kv_head_stride count
 * elements as before), and the value of an element of KV head c is k_scale[c] * e4m3(byte)
 * (v_scale[c] for V).  k_scale_host, v_scale_host: host [Hkv], finite and > 0.  Q, O, lse,
 * workspace, lengths, offsets, window and the result are as for yoco_xattn_decode (Q and O stay
 * bf16); |Q| must stay below 65504, it is widened to fp16 for the products.  d = 128 only,
 * Hkv <= 64.  Half the bytes per key are streamed, so the same bandwidth serves twice the keys. */
int32_t yoco_xattn_decode_fp8(const yoco_xattn_shape* shape, const void* Q, const void* K8, const void* V8,
                              const float* k_scale_host, const float* v_scale_host,
                              const int32_t* cu_kv_host, const int32_t* kv_len_host, void* O, float* lse,
                              void* workspace, size_t workspace_bytes, void* stream);

/* The multi-token path over the same 8-bit cache (arguments as yoco_xattn_decode_fp8, any T >= 1): a
 * prefill or verification chunk against a cache written by yoco_kv_append_fp8.  The bytes are widened
 * to fp16 inside the kernel (exact), Q and P are rounded to fp16 (|Q| < 65504) and the products run on
 * the tensor cores as fp16 x fp16 with fp32 accumulation.  d = 128 only, Hkv <= 64.  The workspace is
 * sized by yoco_xattn_workspace_size_chunk_fp8 (this path always plans two 128-row tiles per CTA, so the
 * size can differ from that of yoco_xattn_chunk for small T). */
int32_t yoco_xattn_chunk_fp8(const yoco_xattn_shape* shape, const void* Q, const void* K8, const void* V8,
                             const float* k_scale_host, const float* v_scale_host,
                             const int32_t* cu_kv_host, const int32_t* kv_len_host, void* O, float* lse,
                             void* workspace, size_t workspace_bytes, void* stream);
int32_t yoco_xattn_workspace_size_chunk_fp8(const yoco_xattn_shape* shape, const int32_t* kv_len_host,
                                            int32_t sm_count, size_t* bytes);

/* (No counterpart in the paper.)  The same merge for pieces laid out piece-major: part_o [S, rows, d], part_lse [S, rows] -- what
 * an all-gather over S ranks leaves when every rank contributes its [rows, d] partial result and
 * its [rows] log-sum-exp.  Otherwise as yoco_xattn_combine. */
int32_t yoco_xattn_combine_gathered(int64_t rows, int32_t S, int32_t d, const float* part_o,
                                    const float* part_lse, void* O, float* lse, void* stream);

/* Decode over ONE SHARD of the keys, for key-range sharding of a long cache across GPUs (the
 * K^, V^ of Section 2.2 split along the sequence, as the chunk-parallel prefill of Appendix A leaves
 * them before its all-gather).  K, V, cu_kv_host, kv_len_host describe the keys this GPU holds (an
 * ordinary packed cache, kv_len[i] may be 0); the result is the attention over those keys only:
 *   part_o   [B*Hq*T, d] fp32, normalised over the shard's keys (0 where the shard holds nothing a row sees)
 *   part_lse [B*Hq*T]    fp32, natural-log sum of exp(score) over the shard's keys (-inf if none)
 * Exchanging (part_o, part_lse) between the shards and merging them with
 * yoco_xattn_combine_gathered gives exactly softmax(QK^T)V over the whole cache (the log-sum-exp
 * merge is algebraically exact).  Workspace as for yoco_xattn_decode.  All pointers device unless
 * marked host.
 *
 * yoco_xattn_decode_partial knows nothing of where the shard sits in the sequence and therefore
 * requires T = 1 and no window: with one query row per head every key of a shard is visible
 * whichever shard holds the row's own position.
 * The _at forms take the shard's place: key_offset_host[i] = index, in sequence i, of the first key
 * held here, kv_total_host[i] = N_i of the whole sequence (host [B] each; key_offset + kv_len <=
 * kv_total).  Query row t then sits at position N_i - T + t of the whole sequence and the causal
 * rule and the window of shape->window apply to whole-sequence key positions, so any T and any
 * window work: decode_partial_at for G*T <= 16 rows per KV head, chunk_partial_at (the tensor-core
 * path) for any T.  Their workspace is sized by yoco_xattn_workspace_size_at. */
int32_t yoco_xattn_decode_partial(const yoco_xattn_shape* shape, const void* Q, const void* K,
                                  const void* V, const int32_t* cu_kv_host, const int32_t* kv_len_host,
                                  float* part_o, float* part_lse, void* workspace,
                                  size_t workspace_bytes, void* stream);
int32_t yoco_xattn_decode_partial_at(const yoco_xattn_shape* shape, const void* Q, const void* K,
                                     const void* V, const int32_t* cu_kv_host, const int32_t* kv_len_host,
                                     const int32_t* key_offset_host, const int32_t* kv_total_host,
                                     float* part_o, float* part_lse, void* workspace,
                                     size_t workspace_bytes, void* stream);
int32_t yoco_xattn_chunk_partial_at(const yoco_xattn_shape* shape, const void* Q, const void* K,
                                    const void* V, const int32_t* cu_kv_host, const int32_t* kv_len_host,
                                    const int32_t* key_offset_host, const int32_t* kv_total_host,
                                    float* part_o, float* part_lse, void* workspace,
                                    size_t workspace_bytes, void* stream);
/* (No counterpart in the paper.)  yoco_xattn_plan and yoco_xattn_workspace_size for a shard at a given
 * place (arguments as above): only the keys that some row of the call sees are planned. */
int32_t yoco_xattn_plan_at(const yoco_xattn_shape* shape, const int32_t* kv_len_host,
                           const int32_t* key_offset_host, const int32_t* kv_total_host, int32_t sm_count,
                           int32_t mode, yoco_xattn_plan_info* info, yoco_xattn_segment* segments_out,
                           int32_t capacity);
int32_t yoco_xattn_workspace_size_at(const yoco_xattn_shape* shape, const int32_t* kv_len_host,
                                     const int32_t* key_offset_host, const int32_t* kv_total_host,
                                     int32_t sm_count, int32_t mode, size_t* bytes);

/* ---- Writing the cache (Section 2.2, first cross-decoder equation) -------------------------
 *   K^ = LN(X) W_K,  V^ = LN(X) W_V,  LN = RMSNorm (Section 2.1), no bias:
 *   LN(x) = x * g / sqrt(mean_k(x_k^2) + eps)
 * X holds the self-decoder's output for the T new tokens of every sequence; the rows produced are
 * stored at positions [N_i - T, N_i) of the packed head-major caches described above, where the
 * attention calls of the cross-decoder layers then find them (kv_len counts them already). */
typedef struct yoco_kv_append_shape {
    int32_t B;               /* sequences (<= 512)                                        */
    int32_t Hkv;             /* KV heads; Hkv * d must be a multiple of 128               */
    int32_t d;               /* head dimension: 64 or 128                                 */
    int32_t T;               /* new tokens per sequence                                   */
    int32_t d_model;         /* width of X; multiple of 128                               */
    float   eps;             /* >= 0, used as given (the paper prints none; 1e-6 is usual) */
    int64_t kv_head_stride;  /* as in yoco_xattn_shape                                    */
} yoco_kv_append_shape;

/* (Section 2.1's RMSNorm as used by Section 2.2's first equation; the folding itself has no
 * counterpart in the paper.)  Folds the RMSNorm gain into a projection weight once per model (weights do not change between
 * calls):  Wg[k, n] = g[k] * W[k, n], one rounding to bf16.  g [d_model], W and Wg [d_model, n_out]
 * row-major bf16, all device; Wg may not alias W. */
int32_t yoco_kv_fold_gain(int64_t d_model, int64_t n_out, const void* g, const void* W, void* Wg,
                          void* stream);

/* Section 2.2, first cross-decoder equation.  Computes the new cache rows and stores them.  X [B*T, d_model] bf16 (sequence-major, the T
 * tokens of a sequence consecutive); Wgk, Wgv [d_model, Hkv*d] bf16 = gain-folded W_K, W_V (see
 * yoco_kv_fold_gain); K, V: the packed caches (device, written in place, 16-byte aligned);
 * cu_kv_host [B+1] or NULL (tight packing), kv_len_host [B]: host, N_i >= T including the new
 * tokens.  Rows outside [N_i - T, N_i) are not touched.  Uses no workspace and only enqueues work.
 * A bounded device-side wait that ran out is reported by yoco_kv_append_status. */
int32_t yoco_kv_append(const yoco_kv_append_shape* shape, const void* X, const void* Wgk, const void* Wgv,
                       void* K, void* V, const int32_t* cu_kv_host, const int32_t* kv_len_host,
                       void* stream);

/* The same step writing an 8-bit cache: every new row is divided by its KV head's scale and stored as
 * FP8 E4M3 bytes (round to nearest even, saturating at +-448) in the byte caches K8, V8 that
 * yoco_xattn_decode_fp8 reads (same packed layout, one byte per element).  k_scale_host, v_scale_host:
 * host [Hkv], finite and > 0, chosen by the caller (for instance the largest magnitude expected / 448);
 * Hkv <= 64.  Otherwise as yoco_kv_append. */
int32_t yoco_kv_append_fp8(const yoco_kv_append_shape* shape, const void* X, const void* Wgk, const void* Wgv,
                           void* K8, void* V8, const float* k_scale_host, const float* v_scale_host,
                           const int32_t* cu_kv_host, const int32_t* kv_len_host, void* stream);

/* (No counterpart in the paper.)  Synchronises `stream`; returns YOCO_OK or YOCO_ERR_TIMEOUT if an
 * append kernel on the current device gave up a wait since the last call of this function (which
 * clears the record).  The _detail form also reports which wait and which CTA (see below). */
int32_t yoco_kv_append_status(void* stream);
int32_t yoco_kv_append_status_detail(void* stream, int32_t* wait_class, int32_t* cta);

/* (No counterpart in the paper.)  Synchronises `stream`, reads the status word that the last
 * decode/chunk call using `workspace` left, returns YOCO_OK or YOCO_ERR_TIMEOUT.  workspace = NULL
 * reads the word of the built-in buffer of yoco_xattn_decode_static on the current device. */
int32_t yoco_xattn_status(const void* workspace, void* stream);

/* What gave up.  The status word is 0, or  wait_class | (cta + 1) << 8  of the first wait that ran
 * out: the kind of wait (YOCO_WAIT_*) and the linear index of the CTA.  yoco_xattn_status_detail
 * reads the word like yoco_xattn_status and decodes it (either output may be NULL; wait_class 0
 * and cta -1 when nothing happened); yoco_xattn_decode_status_word decodes a word the caller holds
 * (pure host).  Both return YOCO_OK or YOCO_ERR_TIMEOUT. */
#define YOCO_WAIT_ITEM_QUEUE 1  /* decode: hand-over of the next work item inside a CTA            */
#define YOCO_WAIT_RING_FULL  2  /* a consumer waiting for a tile copy to land                      */
#define YOCO_WAIT_RING_EMPTY 3  /* the producer waiting for a stage to be released                 */
#define YOCO_WAIT_TENSOR     4  /* tensor-core hand-over: scores ready, P written, product done    */
#define YOCO_WAIT_DRAIN      5  /* on the way out: something already started did not finish        */
#define YOCO_WAIT_MISALIGNED 6  /* shared memory not 1 KB aligned; the kernel did nothing          */
int32_t yoco_xattn_status_detail(const void* workspace, void* stream, int32_t* wait_class, int32_t* cta);
int32_t yoco_xattn_decode_status_word(int32_t word, int32_t* wait_class, int32_t* cta);

/* Self-test of the bounded waits (no counterpart in the paper).  Runs the decode kernel on the given
 * problem (arguments as for yoco_xattn_decode, one work piece per CTA group) with a producer that
 * starts no copy at all and a wait limit of limit_ms milliseconds (1..1000): the first wait for a
 * tile runs out with nothing in flight, the CTAs record it and return, and O is left undefined.
 * Afterwards yoco_xattn_status(workspace) must report YOCO_ERR_TIMEOUT with YOCO_WAIT_RING_FULL, and
 * the next ordinary call on the same device and workspace must work.  Nothing faults, traps or
 * waits without a limit. */
int32_t yoco_xattn_selftest_wait_expiry(const yoco_xattn_shape* shape, const void* Q, const void* K,
                                        const void* V, const int32_t* cu_kv_host, const int32_t* kv_len_host,
                                        void* O, void* workspace, size_t workspace_bytes, int32_t limit_ms,
                                        void* stream);
/* The same for the decode kernel of the 8-bit cache (arguments as for yoco_xattn_decode_fp8; no
 * counterpart in the paper).  Its consumer warps take every fourth tile and first wait for the
 * producer to have armed their tile; with a producer that arms nothing that is the wait that runs
 * out, so the status reads YOCO_ERR_TIMEOUT with YOCO_WAIT_ITEM_QUEUE. */
int32_t yoco_xattn_selftest_wait_expiry_fp8(const yoco_xattn_shape* shape, const void* Q, const void* K8,
                                            const void* V8, const float* k_scale_host, const float* v_scale_host,
                                            const int32_t* cu_kv_host, const int32_t* kv_len_host, void* O,
                                            void* workspace, size_t workspace_bytes, int32_t limit_ms,
                                            void* stream);

/* Measurement aid (no counterpart in the paper).  After yoco_xattn_profile_enable(n), each of
 * the next n decode/chunk calls records a CUDA event pair on its stream around the attention
 * kernel alone (not the merge, not the table upload).  yoco_xattn_profile_collect waits for the
 * recorded pairs, writes their durations in milliseconds (at most `capacity`), stores how many
 * in *count and rearms the same n pairs.  enable(0) switches it off and frees the events. */
int32_t yoco_xattn_profile_enable(int32_t max_records);
int32_t yoco_xattn_profile_collect(float* kernel_ms, int32_t capacity, int32_t* count);

/* (No counterpart in the paper.)  Text of an error code. */
const char* yoco_xattn_strerror(int32_t code);

/* (No counterpart in the paper.)  cudaError_t (as int) of the most recent failing CUDA call on this thread, 0 if none. */
int32_t yoco_xattn_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* YOCO_XATTN_H_ */
