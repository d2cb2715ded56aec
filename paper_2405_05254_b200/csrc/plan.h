// Host-side planner and the device-visible work tables shared by the kernels.
//
// The split-count / tile heuristic: all (sequence, KV head) streams are laid end to end
// in units of key tiles and the resulting flat range is cut into equal contiguous pieces,
// one per CTA group, so that every group streams the same number of K/V bytes and the
// whole grid finishes together in a single wave.
#pragma once

#include <cstddef>
#include <cstdint>
#include <vector>

#include "yoco_xattn.h"

namespace yoco {

constexpr int kDecodeTileN = 64;      // keys per shared-memory stage of the decode kernel
constexpr int kDecodeTileM = 16;      // query rows of one mma.sync tile
constexpr int kDecodeGroupsPerSm = 2; // resident decode CTAs per SM
constexpr int kChunkTileN = 128;      // keys per tcgen05 tile
constexpr int kChunkTileM = 128;      // query rows per tcgen05 tile
constexpr int kChunkPairTileM = 256;  // rows per CTA when a stream has more than 128 rows: two tiles
                                      // that share every K/V tile in shared memory
constexpr int kWorkspaceHeaderBytes = 256;
constexpr int kWorkCounterOffset = 64;  // byte offset of the decode kernel's work counter in the header

// ---- pieces of a decode group ---------------------------------------------------------------
// SMs do not all stream at the same rate (their share of the memory fabric differs with their
// place on the die), so equal static shares leave the fast ones idle at the end.  With R > 1 a
// group's tile range is cut into R pieces of decreasing size; piece 0 is taken by the group's own
// CTA, the rest are handed out in order to whichever CTA is free.  The pieces are fixed by the plan
// (integers only), so the result does not depend on who ran what.
constexpr int kMaxSubItems = 4;

#ifdef __CUDACC__
#define YOCO_HD __host__ __device__
#else
#define YOCO_HD
#endif
// First tile (inside a group of n tiles) of piece r of R, r = 0..R; R in {1, 2, 4}.
YOCO_HD inline int64_t sub_bound(int64_t n, int R, int r) {
    // cumulative shares in 64ths: a large first piece, then smaller and smaller ones
    const unsigned c4 = 0x403D362Cu;                       // 44 54 61 64
    if (r <= 0) return 0;
    if (r >= R) return n;
    const int c = R == 4 ? (int)((c4 >> (8 * (r - 1))) & 0xFF) : 52;   // R == 2: 52 | 12
    return n * c / 64;
}
#undef YOCO_HD

// Pieces per group for a decode plan whose groups hold `tiles_per_group` key tiles on average.
// (Measured on B200, 32 query heads over 8 KV heads: two pieces pay from 128K keys per sequence,
// four from 256K; eight gained nothing over four at 1M and made the merge longer.)
inline int choose_sub_items(int64_t tiles_per_group, int max_sub) {
    int R = tiles_per_group >= 96 ? 4 : tiles_per_group >= 40 ? 2 : 1;
    while (R > max_sub) R /= 2;
    return R < 1 ? 1 : R;
}

// One work segment as the kernels read it (10 x int32 = 40 bytes).
struct DevSegment {
    int32_t kv_row0;     // row of key k_begin in the [rows, d] view of the packed K/V buffers
    int32_t k_begin;     // first key of the range inside its sequence
    int32_t k_end;       // one past the last key
    int32_t q_row0;      // first row of this stream in the [B*Hq*T, d] view of Q / O
    int32_t slot;        // partial-result slot
    int32_t n_kv;        // N_i of the sequence
    int32_t stream_nseg; // segments of this stream (1: the kernel writes the final output)
    int32_t stream;      // b * Hkv + c
    int32_t n_full;      // keys (counted from key 0 of this cache) that query row 0 sees: N_i - T + 1 for a
                         // whole cache; for one shard of a key-range-sharded cache the same count minus
                         // the keys held by earlier shards (may be <= 0 or exceed n_kv).  Row t sees n_full + t.
    int32_t pad_;
};
constexpr int kSegmentWords = 10;

struct Plan {
    yoco_xattn_plan_info info{};
    std::vector<yoco_xattn_segment> segments;   // public form
    std::vector<int32_t> table;                  // device blob: segments, group offsets, stream tables
    // offsets in int32 units inside `table`
    int32_t off_segments = 0, off_group_begin = 0, off_stream_base = 0, off_stream_nseg = 0;
    // byte offsets inside the workspace
    int64_t ws_table = 0, ws_part_lse = 0, ws_part_o = 0;
    int64_t kv_rows_extent = 0;                  // rows of the [rows, d] K/V view that may be touched
    int32_t rows_per_stream = 0;                 // G * T
    int32_t sub_items = 1;                       // pieces per group (decode), see sub_bound
    int32_t coarse_segments = 0;                 // entries of the device segment table; partial slots
                                                 // = coarse_segments * sub_items
};

// Returns YOCO_OK or an error code; fills `plan`.  cu_kv_host may be null (tight packing).
// max_sub_items: upper limit of pieces per decode group (1 = every group is one piece).
// eight_bit_cache: the plan is for an 8-bit cache.  Chunk plans then use the two-row-tile CTA
// (kChunkPairTileM) whatever G*T is (the 8-bit cache is read by that kernel only); decode plans choose
// the pieces per group as for half as many tiles (a tile is half the bytes, and the pieces pay by bytes:
// measured at 55 tiles per group, one piece 51.0 us, two 52.9 us).
// key_offset_host / kv_total_host (both null, or both [B]): the cache described by kv_len_host is
// keys [key_offset[i], key_offset[i] + kv_len[i]) of a sequence of kv_total[i] keys; the causal and
// window masks then use the rows' positions in the whole sequence.
int32_t make_plan(const yoco_xattn_shape& s, const int32_t* cu_kv_host, const int32_t* kv_len_host,
                  int32_t sm_count, int32_t mode, Plan& plan, int32_t max_sub_items = kMaxSubItems,
                  const int32_t* key_offset_host = nullptr, const int32_t* kv_total_host = nullptr,
                  bool eight_bit_cache = false);

int32_t validate_shape(const yoco_xattn_shape& s, int32_t mode);
// Lengths, head stride and token offsets must describe sequences that do not overlap (pure host).
int32_t validate_layout(const yoco_xattn_shape& s, const int32_t* cu_kv_host, const int32_t* kv_len_host);

}  // namespace yoco
