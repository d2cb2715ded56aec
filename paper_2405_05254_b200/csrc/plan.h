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

// One work segment as the kernels read it (8 x int32 = 32 bytes).
struct DevSegment {
    int32_t kv_row0;     // row of key k_begin in the [rows, d] view of the packed K/V buffers
    int32_t k_begin;     // first key of the range inside its sequence
    int32_t k_end;       // one past the last key
    int32_t q_row0;      // first row of this stream in the [B*Hq*T, d] view of Q / O
    int32_t slot;        // partial-result slot
    int32_t n_kv;        // N_i of the sequence
    int32_t stream_nseg; // segments of this stream (1: the kernel writes the final output)
    int32_t stream;      // b * Hkv + c
};

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
};

// Returns YOCO_OK or an error code; fills `plan`.  cu_kv_host may be null (tight packing).
int32_t make_plan(const yoco_xattn_shape& s, const int32_t* cu_kv_host, const int32_t* kv_len_host,
                  int32_t sm_count, int32_t mode, Plan& plan);

int32_t validate_shape(const yoco_xattn_shape& s, int32_t mode);

}  // namespace yoco
