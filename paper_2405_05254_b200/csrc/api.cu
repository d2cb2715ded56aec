// C ABI of the library: argument checks, plan cache, tensor maps, kernel launches.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstring>
#include <list>
#include <memory>
#include <mutex>

#include "kernels.h"
#include "plan.h"
#include "yoco_xattn.h"

namespace yoco {
namespace {

thread_local int32_t g_last_cuda_error = 0;

int32_t cuda_fail(cudaError_t e) {
    g_last_cuda_error = (int32_t)e;
    return YOCO_ERR_CUDA;
}
#define YOCO_CUDA_TRY(expr)                               \
    do {                                                  \
        cudaError_t e__ = (expr);                         \
        if (e__ != cudaSuccess) return cuda_fail(e__);    \
    } while (0)

// ---- per-device state ---------------------------------------------------------------------
constexpr int kMaxDevices = 64;
struct DeviceState {
    bool ready = false;
    int sm_count = 0;
};
std::mutex g_mutex;
DeviceState g_dev[kMaxDevices];

int32_t device_state(DeviceState** out) {
    int dev = 0;
    YOCO_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return YOCO_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState& st = g_dev[dev];
    if (!st.ready) {
        int major = 0;
        YOCO_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
        if (major != 10) return YOCO_ERR_UNSUPPORTED;   // built for sm_100a only
        YOCO_CUDA_TRY(cudaDeviceGetAttribute(&st.sm_count, cudaDevAttrMultiProcessorCount, dev));
        YOCO_CUDA_TRY(decode_kernel_setup());
        YOCO_CUDA_TRY(chunk_kernel_setup());
        YOCO_CUDA_TRY(chunk_pair_kernel_setup());
        YOCO_CUDA_TRY(kv_append_kernel_setup());
        YOCO_CUDA_TRY(decode_fp8_kernel_setup());
        st.ready = true;
    }
    *out = &st;
    return YOCO_OK;
}

// ---- plan cache ---------------------------------------------------------------------------
struct PlanKey {
    yoco_xattn_shape shape;
    int32_t sm_count, mode, max_sub, eight_bit;
    std::vector<int32_t> lens, cu, key_off, totals;
    bool operator==(const PlanKey& o) const {
        return std::memcmp(&shape, &o.shape, sizeof shape) == 0 && sm_count == o.sm_count &&
               mode == o.mode && max_sub == o.max_sub && eight_bit == o.eight_bit && lens == o.lens && cu == o.cu &&
               key_off == o.key_off && totals == o.totals;
    }
};
// A cached plan with the launch-ready forms of its tables.
struct ReadyPlan {
    Plan plan;
    std::vector<int32_t> blob;           // workspace image: zeroed header + tables (upload path)
    bool fits_inline = false;            // tables small enough to travel as kernel parameters
    DecodeInlineTables decode_tab;
    CombineInlineTables combine_tab;
};
struct PlanEntry {
    PlanKey key;
    std::shared_ptr<const ReadyPlan> ready;
};
std::list<PlanEntry> g_plans;   // most recently used first
constexpr size_t kPlanCacheEntries = 16;
// Plans whose table upload was recorded into a CUDA graph: the recorded copy reads the plan's host
// image at every replay, so these are never dropped.
std::vector<std::shared_ptr<const ReadyPlan>> g_captured_plans;

// Looks the plan up (most recently used first) or makes it.  The shared pointer keeps the entry
// alive for the caller even if another thread evicts it from the cache meanwhile.
int32_t cached_plan(const yoco_xattn_shape& s, const int32_t* cu, const int32_t* lens, int32_t sm_count,
                    int32_t mode, int32_t max_sub, std::shared_ptr<const ReadyPlan>& out,
                    const int32_t* key_off = nullptr, const int32_t* totals = nullptr, bool eight_bit = false) {
    PlanKey key;
    std::memset(&key.shape, 0, sizeof key.shape);
    key.shape = s;
    key.sm_count = sm_count;
    key.mode = mode;
    key.max_sub = max_sub;
    key.eight_bit = eight_bit ? 1 : 0;
    if (lens) key.lens.assign(lens, lens + s.B);
    if (cu) key.cu.assign(cu, cu + s.B + 1);
    if (key_off) key.key_off.assign(key_off, key_off + s.B);
    if (totals) key.totals.assign(totals, totals + s.B);
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        for (auto it = g_plans.begin(); it != g_plans.end(); ++it)
            if (it->key == key) {
                g_plans.splice(g_plans.begin(), g_plans, it);
                out = g_plans.front().ready;
                return YOCO_OK;
            }
    }
    auto ready = std::make_shared<ReadyPlan>();
    int32_t rc = make_plan(s, cu, lens, sm_count, mode, ready->plan, max_sub, key_off, totals, eight_bit);
    if (rc != YOCO_OK) return rc;
    const Plan& plan = ready->plan;
    ready->blob.assign(kWorkspaceHeaderBytes / 4 + plan.table.size(), 0);
    std::copy(plan.table.begin(), plan.table.end(), ready->blob.begin() + kWorkspaceHeaderBytes / 4);
    ready->fits_inline = mode == YOCO_MODE_DECODE && plan.coarse_segments <= kInlineSegments &&
                         plan.info.num_groups <= kInlineGroups && plan.info.num_streams <= kInlineStreams;
    if (ready->fits_inline) {
        std::memset(&ready->decode_tab, 0, sizeof ready->decode_tab);
        std::memset(&ready->combine_tab, 0, sizeof ready->combine_tab);
        std::memcpy(ready->decode_tab.seg, plan.table.data() + plan.off_segments,
                    (size_t)plan.coarse_segments * sizeof(DevSegment));
        static_assert(sizeof(DecodeInlineTables) + sizeof(DecodeFp8Params) + 2 * sizeof(CUtensorMap) < 32000,
                      "kernel parameter space");
        std::memcpy(ready->decode_tab.group_begin, plan.table.data() + plan.off_group_begin,
                    (size_t)(plan.info.num_groups + 1) * 4);
        std::memcpy(ready->combine_tab.stream_base, plan.table.data() + plan.off_stream_base,
                    (size_t)plan.info.num_streams * 4);
        std::memcpy(ready->combine_tab.stream_nseg, plan.table.data() + plan.off_stream_nseg,
                    (size_t)plan.info.num_streams * 4);
    }
    out = ready;
    std::lock_guard<std::mutex> lock(g_mutex);
    g_plans.push_front(PlanEntry{std::move(key), std::move(ready)});
    if (g_plans.size() > kPlanCacheEntries) g_plans.pop_back();
    return YOCO_OK;
}

// ---- tensor maps ----------------------------------------------------------------------------
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                   const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

int32_t get_encoder(EncodeTiledFn* fn) {
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_encode) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        YOCO_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q));
        if (q != cudaDriverEntryPointSuccess || !sym) return cuda_fail(cudaErrorNotSupported);
        g_encode = reinterpret_cast<EncodeTiledFn>(sym);
    }
    *fn = g_encode;
    return YOCO_OK;
}

// A serving loop calls with the same cache pointers and extents step after step: the last few
// encoded maps are kept per host thread, keyed by everything that goes into the encoding.
struct MapKey {
    const void* base;
    int64_t rows;
    int32_t d, box_rows, u8;
    bool operator==(const MapKey& o) const {
        return base == o.base && rows == o.rows && d == o.d && box_rows == o.box_rows && u8 == o.u8;
    }
};
struct MapCache {
    static constexpr int kEntries = 8;
    MapKey key[kEntries];
    CUtensorMap map[kEntries];
    int used = 0, next = 0;
    bool find(const MapKey& k, CUtensorMap* out) const {
        for (int i = 0; i < used; ++i)
            if (key[i] == k) {
                *out = map[i];
                return true;
            }
        return false;
    }
    void put(const MapKey& k, const CUtensorMap& m) {
        key[next] = k;
        map[next] = m;
        next = (next + 1) % kEntries;
        if (used < kEntries) ++used;
    }
};
thread_local MapCache g_maps;

// 2-D bf16 map over a row-major [rows, d] matrix, box {64 channels, box_rows}, 128-byte swizzle.
int32_t make_map_2d(CUtensorMap* map, const void* base, int64_t rows, int32_t d, int32_t box_rows) {
    const MapKey mk{base, rows, d, box_rows, 0};
    if (g_maps.find(mk, map)) return YOCO_OK;
    EncodeTiledFn enc;
    int32_t rc = get_encoder(&enc);
    if (rc != YOCO_OK) return rc;
    cuuint64_t gdim[2] = {(cuuint64_t)d, (cuuint64_t)rows};
    cuuint64_t gstride[1] = {(cuuint64_t)d * 2};
    cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1u, 1u};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride,
                     box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cuda_fail(cudaErrorInvalidValue);
    g_maps.put(mk, *map);
    return YOCO_OK;
}

// 2-D byte map over a row-major [rows, 128] matrix of FP8 values, box {128, box_rows}, 128-byte swizzle.
int32_t make_map_2d_u8(CUtensorMap* map, const void* base, int64_t rows, int32_t box_rows) {
    const MapKey mk{base, rows, 128, box_rows, 1};
    if (g_maps.find(mk, map)) return YOCO_OK;
    EncodeTiledFn enc;
    int32_t rc = get_encoder(&enc);
    if (rc != YOCO_OK) return rc;
    cuuint64_t gdim[2] = {128u, (cuuint64_t)rows};
    cuuint64_t gstride[1] = {128u};
    cuuint32_t box[2] = {128u, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1u, 1u};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), gdim, gstride, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cuda_fail(cudaErrorInvalidValue);
    g_maps.put(mk, *map);
    return YOCO_OK;
}

// per-head scales of an 8-bit cache (host pointers)
struct Fp8Scales {
    const float* k_scale;
    const float* v_scale;
};

// ---- optional per-launch timing of the attention kernel -------------------------------------
struct Profiler {
    std::vector<cudaEvent_t> events;   // pairs: before / after the attention kernel
    int32_t used = 0;                  // pairs recorded so far
} g_prof;

cudaEvent_t prof_event(bool after, bool* active) {
    std::lock_guard<std::mutex> lock(g_mutex);
    const int32_t pairs = (int32_t)g_prof.events.size() / 2;
    if (g_prof.used >= pairs) {
        *active = false;
        return nullptr;
    }
    *active = true;
    cudaEvent_t e = g_prof.events[2 * g_prof.used + (after ? 1 : 0)];
    if (after) ++g_prof.used;
    return e;
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// self-test of the give-up path of the decode kernel (yoco_xattn_selftest_wait_expiry)
struct SelfTest {
    int64_t wait_limit_ns;
};
// where the keys of this call sit in the whole sequences (one shard of a key-range-sharded cache)
struct ShardPos {
    const int32_t* key_offset;   // host [B]
    const int32_t* kv_total;     // host [B]
};

int32_t run(const yoco_xattn_shape* shape, int32_t mode, const void* Q, const void* K, const void* V,
            const int32_t* cu_kv_host, const int32_t* kv_len_host, void* O, float* lse,
            void* workspace, size_t workspace_bytes, void* stream_v, float* part_out = nullptr,
            const Fp8Scales* fp8 = nullptr, int32_t max_sub = kMaxSubItems, const SelfTest* selftest = nullptr,
            const ShardPos* shard = nullptr) {
    // part_out != null: the result is a partial one (fp32 rows + their LSE in `lse`, no bf16 O)
    if (!shape) return YOCO_ERR_INVALID_ARG;
    int32_t rc = validate_shape(*shape, mode);
    if (rc != YOCO_OK) return rc;
    if (shape->B == 0) return YOCO_OK;
    if (!Q || !K || !V || !(O || part_out) || !workspace) return YOCO_ERR_INVALID_ARG;
    if (part_out && (!lse || !aligned(part_out, 16))) return YOCO_ERR_INVALID_ARG;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) ||
        !aligned(workspace, 256) || (lse && !aligned(lse, 4)))
        return YOCO_ERR_INVALID_ARG;
    if ((rc = validate_layout(*shape, cu_kv_host, kv_len_host)) != YOCO_OK) return rc;

    DeviceState* dev = nullptr;
    if ((rc = device_state(&dev)) != YOCO_OK) return rc;

    std::shared_ptr<const ReadyPlan> ready;
    if ((rc = cached_plan(*shape, cu_kv_host, kv_len_host, dev->sm_count, mode, max_sub, ready,
                          shard ? shard->key_offset : nullptr, shard ? shard->kv_total : nullptr,
                          fp8 != nullptr)) != YOCO_OK)
        return rc;
    const Plan& plan = ready->plan;
    if ((int64_t)workspace_bytes < plan.info.workspace_bytes) return YOCO_ERR_WORKSPACE_TOO_SMALL;

    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_v);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const float scale = shape->scale != 0.f ? shape->scale : 1.f / std::sqrt((float)shape->d);

    const bool inline_tables = ready->fits_inline;
    if (inline_tables) {
        // the tables travel as kernel parameters: only the status word has to be cleared
        YOCO_CUDA_TRY(cudaMemsetAsync(ws, 0, kWorkspaceHeaderBytes, stream));
    } else {
        // header (status word = 0) + work tables in one copy.  The source is pageable memory, which
        // the runtime stages before the call returns, so the cache entry may go away afterwards --
        // unless the stream is being recorded into a graph: the recorded copy reads the same host
        // memory again at every replay, so such a plan is kept for the life of the process.
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        YOCO_CUDA_TRY(cudaStreamIsCapturing(stream, &cap));
        if (cap != cudaStreamCaptureStatusNone) {
            std::lock_guard<std::mutex> lock(g_mutex);
            bool kept = false;
            for (const auto& q : g_captured_plans) kept = kept || q == ready;
            if (!kept) g_captured_plans.push_back(ready);
        }
        YOCO_CUDA_TRY(cudaMemcpyAsync(ws, ready->blob.data(), ready->blob.size() * 4, cudaMemcpyHostToDevice,
                                      stream));
    }
    const int32_t* table = reinterpret_cast<const int32_t*>(ws + plan.ws_table);
    float* part_lse = reinterpret_cast<float*>(ws + plan.ws_part_lse);
    float* part_o = reinterpret_cast<float*>(ws + plan.ws_part_o);
    int32_t* status = reinterpret_cast<int32_t*>(ws);

    bool timed = false;   // an event pair was put around the attention kernel of this call
    if (plan.info.num_segments > 0) {
        bool prof = false;
        cudaEvent_t ev = prof_event(false, &prof);
        if (prof) YOCO_CUDA_TRY(cudaEventRecord(ev, stream));
        timed = prof;
        if (mode == YOCO_MODE_DECODE) {
            CUtensorMap tmK, tmV;
            if (fp8) {
                if ((rc = make_map_2d_u8(&tmK, K, plan.kv_rows_extent, kDecodeTileN)) != YOCO_OK) return rc;
                if ((rc = make_map_2d_u8(&tmV, V, plan.kv_rows_extent, kDecodeTileN)) != YOCO_OK) return rc;
            } else {
                if ((rc = make_map_2d(&tmK, K, plan.kv_rows_extent, shape->d, kDecodeTileN)) != YOCO_OK) return rc;
                if ((rc = make_map_2d(&tmV, V, plan.kv_rows_extent, shape->d, kDecodeTileN)) != YOCO_OK) return rc;
            }
            DecodeParams p{};
            p.Q = static_cast<const __nv_bfloat16*>(Q);
            p.O = static_cast<__nv_bfloat16*>(O);
            p.lse = lse;
            p.segments = reinterpret_cast<const DevSegment*>(table + plan.off_segments);
            p.group_begin = table + plan.off_group_begin;
            p.part_o = part_o;
            p.part_lse = part_lse;
            p.status = status;
            p.scale_log2 = scale * 1.4426950408889634f;
            p.T = shape->T;
            p.rows_per_stream = plan.rows_per_stream;
            p.d = shape->d;
            p.window = shape->window;
            p.force_partial = part_out ? 1 : 0;
            p.sub_items = plan.sub_items;
            p.work_counter = reinterpret_cast<int32_t*>(ws + kWorkCounterOffset);
            if (selftest) {
                p.wait_limit_ns = selftest->wait_limit_ns;
                p.selftest_skip_loads = 1;
            }
            if (fp8) {
                DecodeFp8Params p8{};
                p8.base = p;
                p8.Hkv = shape->Hkv;
                for (int c = 0; c < shape->Hkv; ++c) {
                    p8.score_scale_log2[c] = scale * fp8->k_scale[c] * 1.4426950408889634f;
                    p8.v_scale[c] = fp8->v_scale[c];
                }
                YOCO_CUDA_TRY(launch_decode_fp8(p8, tmK, tmV, plan.info.num_groups, stream,
                                                inline_tables ? &ready->decode_tab : nullptr));
            } else {
                YOCO_CUDA_TRY(launch_decode(p, tmK, tmV, plan.info.num_groups, stream,
                                            inline_tables ? &ready->decode_tab : nullptr));
            }
        } else {
            CUtensorMap tmQ, tmK, tmV;
            const int64_t q_rows = (int64_t)shape->B * shape->Hq * shape->T;
            if ((rc = make_map_2d(&tmQ, Q, q_rows, shape->d, kChunkTileM)) != YOCO_OK) return rc;
            if (fp8) {
                if ((rc = make_map_2d_u8(&tmK, K, plan.kv_rows_extent, kChunkTileN)) != YOCO_OK) return rc;
                if ((rc = make_map_2d_u8(&tmV, V, plan.kv_rows_extent, kChunkTileN)) != YOCO_OK) return rc;
            } else {
                if ((rc = make_map_2d(&tmK, K, plan.kv_rows_extent, shape->d, kChunkTileN)) != YOCO_OK) return rc;
                if ((rc = make_map_2d(&tmV, V, plan.kv_rows_extent, shape->d, kChunkTileN)) != YOCO_OK) return rc;
            }
            ChunkParams p{};
            p.O = static_cast<__nv_bfloat16*>(O);
            p.lse = lse;
            p.segments = reinterpret_cast<const DevSegment*>(table + plan.off_segments);
            p.group_begin = table + plan.off_group_begin;
            p.part_o = part_o;
            p.part_lse = part_lse;
            p.status = status;
            p.scale_log2 = scale * 1.4426950408889634f;
            p.T = shape->T;
            p.rows_per_stream = plan.rows_per_stream;
            p.m_tiles = plan.info.m_tiles;
            p.d = shape->d;
            p.window = shape->window;
            p.force_partial = part_out ? 1 : 0;
            if (fp8) {
                ChunkFp8Scales cs{};
                cs.Hkv = shape->Hkv;
                for (int c = 0; c < shape->Hkv; ++c) {
                    cs.score_scale_log2[c] = scale * fp8->k_scale[c] * 1.4426950408889634f;
                    cs.v_scale[c] = fp8->v_scale[c];
                }
                YOCO_CUDA_TRY(launch_chunk_pair(p, tmQ, tmK, tmV, plan.info.num_groups, stream, &cs));
            } else if (plan.info.tile_m == kChunkPairTileM)
                YOCO_CUDA_TRY(launch_chunk_pair(p, tmQ, tmK, tmV, plan.info.num_groups, stream));
            else
                YOCO_CUDA_TRY(launch_chunk(p, tmQ, tmK, tmV, plan.info.num_groups, stream));
        }
        if (prof) {
            ev = prof_event(true, &prof);
            if (prof) YOCO_CUDA_TRY(cudaEventRecord(ev, stream));
        }
    }
    if (plan.info.needs_combine || part_out) {
        CombineParams c{};
        c.rows = (int64_t)shape->B * shape->Hq * shape->T;
        c.d = shape->d;
        c.S = 0;
        c.Hq = shape->Hq;
        c.Hkv = shape->Hkv;
        c.T = shape->T;
        c.rows_per_stream = plan.rows_per_stream;
        c.max_pieces = plan.info.max_splits;
        c.sub_items = plan.sub_items;
        c.stream_base = table + plan.off_stream_base;
        c.stream_nseg = table + plan.off_stream_nseg;
        c.part_o = part_o;
        c.part_lse = part_lse;
        c.O = part_out ? nullptr : static_cast<__nv_bfloat16*>(O);
        c.lse = lse;
        c.O_f32 = part_out;
        c.merge_unsplit = part_out ? 1 : 0;
        // directly behind the attention kernel (no event in between): its launch may overlap
        // that kernel's tail
        const bool chained = plan.info.num_segments > 0 && !timed;
        YOCO_CUDA_TRY(launch_combine(c, stream, inline_tables ? &ready->combine_tab : nullptr, chained));
    }
    return YOCO_OK;
}


// ---- built-in scratch for callers that cannot allocate -------------------------------------
// Lives in every GPU that loads this library until the process exits.  In host code the
// name below is only a handle; the device address comes from cudaGetSymbolAddress.
constexpr size_t kStaticScratchBytes = 4u << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
void* g_static_scratch_addr[kMaxDevices] = {};

int32_t static_scratch_address(void** out) {
    int dev = 0;
    YOCO_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return YOCO_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_static_scratch_addr[dev]) {
        void* ptr = nullptr;
        YOCO_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));   // address on the current device
        if (!ptr) return cuda_fail(cudaErrorInvalidSymbol);
        g_static_scratch_addr[dev] = ptr;
    }
    *out = g_static_scratch_addr[dev];
    return YOCO_OK;
}

}  // namespace
}  // namespace yoco

using namespace yoco;

extern "C" {

int32_t yoco_xattn_plan(const yoco_xattn_shape* shape, const int32_t* kv_len_host, int32_t sm_count,
                        int32_t mode, yoco_xattn_plan_info* info, yoco_xattn_segment* segments_out,
                        int32_t capacity) {
    return yoco_xattn_plan_at(shape, kv_len_host, nullptr, nullptr, sm_count, mode, info, segments_out, capacity);
}

int32_t yoco_xattn_plan_at(const yoco_xattn_shape* shape, const int32_t* kv_len_host, const int32_t* key_offset_host,
                           const int32_t* kv_total_host, int32_t sm_count, int32_t mode, yoco_xattn_plan_info* info,
                           yoco_xattn_segment* segments_out, int32_t capacity) {
    if (!shape || !info || capacity < 0 || (capacity > 0 && !segments_out)) return YOCO_ERR_INVALID_ARG;
    Plan plan;
    int32_t rc = make_plan(*shape, nullptr, kv_len_host, sm_count, mode, plan, kMaxSubItems, key_offset_host,
                           kv_total_host);
    if (rc != YOCO_OK) return rc;
    *info = plan.info;
    const int32_t n = std::min<int32_t>(capacity, (int32_t)plan.segments.size());
    for (int32_t k = 0; k < n; ++k) segments_out[k] = plan.segments[k];
    return YOCO_OK;
}

int64_t yoco_xattn_sub_bound(int64_t n_tiles, int32_t sub_items, int32_t r) {
    if (n_tiles < 0 || (sub_items != 1 && sub_items != 2 && sub_items != 4)) return -1;
    return sub_bound(n_tiles, sub_items, r);
}

int32_t yoco_xattn_workspace_size(const yoco_xattn_shape* shape, const int32_t* kv_len_host,
                                  int32_t sm_count, int32_t mode, size_t* bytes) {
    return yoco_xattn_workspace_size_at(shape, kv_len_host, nullptr, nullptr, sm_count, mode, bytes);
}

int32_t yoco_xattn_workspace_size_at(const yoco_xattn_shape* shape, const int32_t* kv_len_host,
                                     const int32_t* key_offset_host, const int32_t* kv_total_host,
                                     int32_t sm_count, int32_t mode, size_t* bytes) {
    if (!shape || !bytes || sm_count < 0) return YOCO_ERR_INVALID_ARG;
    if (sm_count == 0) {
        int32_t rc = validate_shape(*shape, mode);
        if (rc != YOCO_OK) return rc;
        DeviceState* dev = nullptr;
        if ((rc = device_state(&dev)) != YOCO_OK) return rc;
        sm_count = dev->sm_count;
    }
    Plan plan;
    int32_t rc = make_plan(*shape, nullptr, kv_len_host, sm_count, mode, plan, kMaxSubItems, key_offset_host,
                           kv_total_host);
    if (rc != YOCO_OK) return rc;
    *bytes = (size_t)plan.info.workspace_bytes;
    return YOCO_OK;
}

int32_t yoco_xattn_decode(const yoco_xattn_shape* shape, const void* Q, const void* K, const void* V,
                          const int32_t* cu_kv_host, const int32_t* kv_len_host, void* O, float* lse,
                          void* workspace, size_t workspace_bytes, void* stream) {
    return run(shape, YOCO_MODE_DECODE, Q, K, V, cu_kv_host, kv_len_host, O, lse, workspace,
               workspace_bytes, stream);
}

int32_t yoco_xattn_decode_static(const yoco_xattn_shape* shape, const void* Q, const void* K,
                                 const void* V, const int32_t* cu_kv_host, const int32_t* kv_len_host,
                                 void* O, float* lse, void* stream) {
    if (!shape) return YOCO_ERR_INVALID_ARG;
    int32_t rc = validate_shape(*shape, YOCO_MODE_DECODE);
    if (rc != YOCO_OK) return rc;
    if (shape->B == 0) return YOCO_OK;
    // size check first, on the host: nothing is enqueued for a problem that does not fit
    DeviceState* dev = nullptr;
    if ((rc = device_state(&dev)) != YOCO_OK) return rc;
    // one piece per group: the fixed buffer is sized for that
    std::shared_ptr<const ReadyPlan> ready;
    if ((rc = cached_plan(*shape, cu_kv_host, kv_len_host, dev->sm_count, YOCO_MODE_DECODE, 1, ready)) != YOCO_OK)
        return rc;
    if ((size_t)ready->plan.info.workspace_bytes > kStaticScratchBytes) return YOCO_ERR_STATIC_SCRATCH_EXCEEDED;
    void* scratch = nullptr;
    if ((rc = static_scratch_address(&scratch)) != YOCO_OK) return rc;
    return run(shape, YOCO_MODE_DECODE, Q, K, V, cu_kv_host, kv_len_host, O, lse, scratch,
               kStaticScratchBytes, stream, nullptr, nullptr, 1);
}

int32_t yoco_xattn_static_scratch_bytes(void) { return (int32_t)kStaticScratchBytes; }

int32_t yoco_xattn_chunk(const yoco_xattn_shape* shape, const void* Q, const void* K, const void* V,
                         const int32_t* cu_kv_host, const int32_t* kv_len_host, void* O, float* lse,
                         void* workspace, size_t workspace_bytes, void* stream) {
    return run(shape, YOCO_MODE_CHUNK, Q, K, V, cu_kv_host, kv_len_host, O, lse, workspace,
               workspace_bytes, stream);
}

namespace {
int32_t combine_public(int64_t rows, int32_t S, int32_t d, const float* part_o, const float* part_lse, void* O,
                       float* lse, void* stream, int32_t piece_major) {
    if (rows < 0 || S <= 0 || d <= 0) return YOCO_ERR_INVALID_ARG;
    if (d % 8 != 0 || d > 256) return YOCO_ERR_UNSUPPORTED;
    if (rows == 0) return YOCO_OK;
    if (!part_o || !part_lse || !O) return YOCO_ERR_INVALID_ARG;
    if (!aligned(part_o, 16) || !aligned(part_lse, 4) || !aligned(O, 16)) return YOCO_ERR_INVALID_ARG;
    CombineParams c{};
    c.rows = rows;
    c.d = d;
    c.S = S;
    c.max_pieces = S;
    c.stream_base = nullptr;
    c.stream_nseg = nullptr;
    c.part_o = part_o;
    c.part_lse = part_lse;
    c.O = static_cast<__nv_bfloat16*>(O);
    c.lse = lse;
    c.piece_major = piece_major;
    YOCO_CUDA_TRY(launch_combine(c, reinterpret_cast<cudaStream_t>(stream)));
    return YOCO_OK;
}
}  // namespace

int32_t yoco_xattn_combine(int64_t rows, int32_t S, int32_t d, const float* part_o,
                           const float* part_lse, void* O, float* lse, void* stream) {
    return combine_public(rows, S, d, part_o, part_lse, O, lse, stream, 0);
}

int32_t yoco_xattn_combine_gathered(int64_t rows, int32_t S, int32_t d, const float* part_o,
                                    const float* part_lse, void* O, float* lse, void* stream) {
    return combine_public(rows, S, d, part_o, part_lse, O, lse, stream, 1);
}

namespace {
int32_t partial_impl(int32_t mode, const yoco_xattn_shape* shape, const void* Q, const void* K, const void* V,
                     const int32_t* cu_kv_host, const int32_t* kv_len_host, const int32_t* key_offset_host,
                     const int32_t* kv_total_host, float* part_o, float* part_lse, void* workspace,
                     size_t workspace_bytes, void* stream) {
    if (!shape || !part_o || !part_lse) return YOCO_ERR_INVALID_ARG;
    if ((key_offset_host == nullptr) != (kv_total_host == nullptr)) return YOCO_ERR_INVALID_ARG;
    // Without the shard's place in the sequence only T = 1 without a window can be answered: then every
    // key of a shard is visible whatever follows it on other shards.
    if (!key_offset_host && (shape->T != 1 || shape->window != 0)) return YOCO_ERR_UNSUPPORTED;
    if (key_offset_host && !kv_len_host) return YOCO_ERR_INVALID_ARG;
    const ShardPos pos{key_offset_host, kv_total_host};
    return run(shape, mode, Q, K, V, cu_kv_host, kv_len_host, nullptr, part_lse, workspace, workspace_bytes, stream,
               part_o, nullptr, kMaxSubItems, nullptr, key_offset_host ? &pos : nullptr);
}
}  // namespace

int32_t yoco_xattn_decode_partial(const yoco_xattn_shape* shape, const void* Q, const void* K, const void* V,
                                  const int32_t* cu_kv_host, const int32_t* kv_len_host, float* part_o,
                                  float* part_lse, void* workspace, size_t workspace_bytes, void* stream) {
    return partial_impl(YOCO_MODE_DECODE, shape, Q, K, V, cu_kv_host, kv_len_host, nullptr, nullptr, part_o, part_lse,
                        workspace, workspace_bytes, stream);
}

int32_t yoco_xattn_decode_partial_at(const yoco_xattn_shape* shape, const void* Q, const void* K, const void* V,
                                     const int32_t* cu_kv_host, const int32_t* kv_len_host,
                                     const int32_t* key_offset_host, const int32_t* kv_total_host, float* part_o,
                                     float* part_lse, void* workspace, size_t workspace_bytes, void* stream) {
    if (!key_offset_host || !kv_total_host) return YOCO_ERR_INVALID_ARG;
    return partial_impl(YOCO_MODE_DECODE, shape, Q, K, V, cu_kv_host, kv_len_host, key_offset_host, kv_total_host,
                        part_o, part_lse, workspace, workspace_bytes, stream);
}

int32_t yoco_xattn_chunk_partial_at(const yoco_xattn_shape* shape, const void* Q, const void* K, const void* V,
                                    const int32_t* cu_kv_host, const int32_t* kv_len_host,
                                    const int32_t* key_offset_host, const int32_t* kv_total_host, float* part_o,
                                    float* part_lse, void* workspace, size_t workspace_bytes, void* stream) {
    if (!key_offset_host || !kv_total_host) return YOCO_ERR_INVALID_ARG;
    return partial_impl(YOCO_MODE_CHUNK, shape, Q, K, V, cu_kv_host, kv_len_host, key_offset_host, kv_total_host,
                        part_o, part_lse, workspace, workspace_bytes, stream);
}

int32_t yoco_xattn_decode_fp8(const yoco_xattn_shape* shape, const void* Q, const void* K8, const void* V8,
                              const float* k_scale_host, const float* v_scale_host, const int32_t* cu_kv_host,
                              const int32_t* kv_len_host, void* O, float* lse, void* workspace,
                              size_t workspace_bytes, void* stream) {
    if (!shape || !k_scale_host || !v_scale_host) return YOCO_ERR_INVALID_ARG;
    if (shape->d != 128 || shape->Hkv > kFp8MaxHeads) return YOCO_ERR_UNSUPPORTED;
    for (int c = 0; c < shape->Hkv; ++c)
        if (!(k_scale_host[c] > 0.f) || !(v_scale_host[c] > 0.f) || !std::isfinite(k_scale_host[c]) ||
            !std::isfinite(v_scale_host[c]))
            return YOCO_ERR_INVALID_ARG;
    const Fp8Scales sc{k_scale_host, v_scale_host};
    return run(shape, YOCO_MODE_DECODE, Q, K8, V8, cu_kv_host, kv_len_host, O, lse, workspace, workspace_bytes,
               stream, nullptr, &sc);
}

int32_t yoco_xattn_chunk_fp8(const yoco_xattn_shape* shape, const void* Q, const void* K8, const void* V8,
                             const float* k_scale_host, const float* v_scale_host, const int32_t* cu_kv_host,
                             const int32_t* kv_len_host, void* O, float* lse, void* workspace,
                             size_t workspace_bytes, void* stream) {
    if (!shape || !k_scale_host || !v_scale_host) return YOCO_ERR_INVALID_ARG;
    if (shape->d != 128 || shape->Hkv > kFp8MaxHeads) return YOCO_ERR_UNSUPPORTED;
    for (int c = 0; c < shape->Hkv; ++c)
        if (!(k_scale_host[c] > 0.f) || !(v_scale_host[c] > 0.f) || !std::isfinite(k_scale_host[c]) ||
            !std::isfinite(v_scale_host[c]))
            return YOCO_ERR_INVALID_ARG;
    const Fp8Scales sc{k_scale_host, v_scale_host};
    return run(shape, YOCO_MODE_CHUNK, Q, K8, V8, cu_kv_host, kv_len_host, O, lse, workspace, workspace_bytes,
               stream, nullptr, &sc);
}

int32_t yoco_xattn_workspace_size_chunk_fp8(const yoco_xattn_shape* shape, const int32_t* kv_len_host,
                                            int32_t sm_count, size_t* bytes) {
    if (!shape || !bytes || sm_count < 0) return YOCO_ERR_INVALID_ARG;
    if (sm_count == 0) {
        int32_t rc = validate_shape(*shape, YOCO_MODE_CHUNK);
        if (rc != YOCO_OK) return rc;
        DeviceState* dev = nullptr;
        if ((rc = device_state(&dev)) != YOCO_OK) return rc;
        sm_count = dev->sm_count;
    }
    Plan plan;
    int32_t rc = make_plan(*shape, nullptr, kv_len_host, sm_count, YOCO_MODE_CHUNK, plan, kMaxSubItems, nullptr, nullptr,
                           true);
    if (rc != YOCO_OK) return rc;
    *bytes = (size_t)plan.info.workspace_bytes;
    return YOCO_OK;
}

int32_t yoco_kv_fold_gain(int64_t d_model, int64_t n_out, const void* g, const void* W, void* Wg, void* stream) {
    if (d_model < 0 || n_out < 0) return YOCO_ERR_INVALID_ARG;
    if (d_model == 0 || n_out == 0) return YOCO_OK;
    if (!g || !W || !Wg || W == Wg) return YOCO_ERR_INVALID_ARG;
    YOCO_CUDA_TRY(launch_fold_gain(static_cast<const __nv_bfloat16*>(g), static_cast<const __nv_bfloat16*>(W),
                                   static_cast<__nv_bfloat16*>(Wg), d_model, n_out,
                                   reinterpret_cast<cudaStream_t>(stream)));
    return YOCO_OK;
}

namespace {
int32_t kv_append_impl(const yoco_kv_append_shape* shape, const void* X, const void* Wgk, const void* Wgv, void* K,
                       void* V, const float* k_scale_host, const float* v_scale_host, bool fp8,
                       const int32_t* cu_kv_host, const int32_t* kv_len_host, void* stream) {
    if (!shape) return YOCO_ERR_INVALID_ARG;
    const yoco_kv_append_shape& s = *shape;
    if (s.B < 0 || s.Hkv <= 0 || s.d <= 0 || s.T <= 0 || s.d_model <= 0 || s.kv_head_stride < 0 || !(s.eps >= 0.f))
        return YOCO_ERR_INVALID_ARG;
    if ((s.d != 64 && s.d != 128) || s.d_model % 128 != 0 || (s.Hkv * s.d) % 128 != 0 ||
        s.kv_head_stride % s.d != 0 || s.B > kAppendMaxSequences || (int64_t)s.B * s.T >= (1ll << 31))
        return YOCO_ERR_UNSUPPORTED;
    if (s.B == 0) return YOCO_OK;
    if (!X || !Wgk || !Wgv || !K || !V || !kv_len_host) return YOCO_ERR_INVALID_ARG;
    if (!aligned(X, 16) || !aligned(Wgk, 16) || !aligned(Wgv, 16) || !aligned(K, 16) || !aligned(V, 16))
        return YOCO_ERR_INVALID_ARG;
    KvAppendTables tab;
    std::memset(&tab, 0, sizeof tab);
    int64_t tok = 0;
    for (int i = 0; i < s.B; ++i) {
        const int64_t n = kv_len_host[i];
        if (n < s.T) return YOCO_ERR_INVALID_ARG;
        const int64_t head_rows = s.kv_head_stride ? s.kv_head_stride / s.d : n;
        if (head_rows < n) return YOCO_ERR_INVALID_ARG;
        if (cu_kv_host) {
            if (cu_kv_host[i] < 0 || cu_kv_host[i + 1] < cu_kv_host[i]) return YOCO_ERR_INVALID_ARG;
            // the rows written for sequence i may not reach into the next sequence's heads
            if ((int64_t)cu_kv_host[i + 1] - cu_kv_host[i] < head_rows) return YOCO_ERR_INVALID_ARG;
            tok = cu_kv_host[i];
        }
        const int64_t row0 = tok * s.Hkv + (n - s.T);
        if (row0 + (int64_t)(s.Hkv - 1) * head_rows + s.T >= (1ll << 31)) return YOCO_ERR_UNSUPPORTED;
        tab.row0[i] = (int32_t)row0;
        tab.head_rows[i] = (int32_t)head_rows;
        if (!cu_kv_host) tok += head_rows;
    }
    DeviceState* dev = nullptr;
    int32_t rc = device_state(&dev);
    if (rc != YOCO_OK) return rc;
    KvAppendParams p{};
    p.X = static_cast<const __nv_bfloat16*>(X);
    p.K = static_cast<__nv_bfloat16*>(K);
    p.V = static_cast<__nv_bfloat16*>(V);
    p.M = s.B * s.T;
    p.T = s.T;
    p.d = s.d;
    p.d_model = s.d_model;
    p.n_half = s.Hkv * s.d;
    p.eps = s.eps;
    CUtensorMap tmX, tmWk, tmWv;
    if ((rc = make_map_2d(&tmX, X, p.M, s.d_model, 128)) != YOCO_OK) return rc;
    if ((rc = make_map_2d(&tmWk, Wgk, s.d_model, p.n_half, 128)) != YOCO_OK) return rc;
    if ((rc = make_map_2d(&tmWv, Wgv, s.d_model, p.n_half, 128)) != YOCO_OK) return rc;
    KvAppendScales sc{};
    if (fp8) {
        if (!k_scale_host || !v_scale_host) return YOCO_ERR_INVALID_ARG;
        if (s.Hkv > kFp8MaxHeads) return YOCO_ERR_UNSUPPORTED;
        for (int c = 0; c < s.Hkv; ++c) {
            if (!(k_scale_host[c] > 0.f) || !(v_scale_host[c] > 0.f) || !std::isfinite(k_scale_host[c]) ||
                !std::isfinite(v_scale_host[c]))
                return YOCO_ERR_INVALID_ARG;
            sc.inv_k[c] = 1.f / k_scale_host[c];
            sc.inv_v[c] = 1.f / v_scale_host[c];
        }
    }
    YOCO_CUDA_TRY(launch_kv_append(p, tab, tmX, tmWk, tmWv, reinterpret_cast<cudaStream_t>(stream), fp8 ? &sc : nullptr));
    return YOCO_OK;
}
}  // namespace

int32_t yoco_kv_append(const yoco_kv_append_shape* shape, const void* X, const void* Wgk, const void* Wgv,
                       void* K, void* V, const int32_t* cu_kv_host, const int32_t* kv_len_host, void* stream) {
    return kv_append_impl(shape, X, Wgk, Wgv, K, V, nullptr, nullptr, false, cu_kv_host, kv_len_host, stream);
}

int32_t yoco_kv_append_fp8(const yoco_kv_append_shape* shape, const void* X, const void* Wgk, const void* Wgv,
                           void* K8, void* V8, const float* k_scale_host, const float* v_scale_host,
                           const int32_t* cu_kv_host, const int32_t* kv_len_host, void* stream) {
    return kv_append_impl(shape, X, Wgk, Wgv, K8, V8, k_scale_host, v_scale_host, true, cu_kv_host, kv_len_host,
                          stream);
}

int32_t yoco_kv_append_status(void* stream) {
    int32_t word = 0;
    YOCO_CUDA_TRY(read_and_clear_kv_append_status(&word, reinterpret_cast<cudaStream_t>(stream)));
    return word == kStatusOk ? YOCO_OK : YOCO_ERR_TIMEOUT;
}

int32_t yoco_kv_append_status_detail(void* stream, int32_t* wait_class, int32_t* cta) {
    int32_t word = 0;
    YOCO_CUDA_TRY(read_and_clear_kv_append_status(&word, reinterpret_cast<cudaStream_t>(stream)));
    return yoco_xattn_decode_status_word(word, wait_class, cta);
}

namespace {
// reads the status word of `workspace`, or of the built-in buffer of the current device when null
int32_t read_status_word(const void* workspace, void* stream, int32_t* word) {
    void* builtin = nullptr;
    if (!workspace) {
        int32_t rc = static_scratch_address(&builtin);
        if (rc != YOCO_OK) return rc;
        workspace = builtin;
    }
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    YOCO_CUDA_TRY(cudaMemcpyAsync(word, workspace, sizeof *word, cudaMemcpyDeviceToHost, s));
    YOCO_CUDA_TRY(cudaStreamSynchronize(s));
    return YOCO_OK;
}
}  // namespace

int32_t yoco_xattn_status(const void* workspace, void* stream) {
    int32_t word = 0;
    int32_t rc = read_status_word(workspace, stream, &word);
    if (rc != YOCO_OK) return rc;
    return word == kStatusOk ? YOCO_OK : YOCO_ERR_TIMEOUT;
}

int32_t yoco_xattn_status_detail(const void* workspace, void* stream, int32_t* wait_class, int32_t* cta) {
    int32_t word = 0;
    int32_t rc = read_status_word(workspace, stream, &word);
    if (rc != YOCO_OK) return rc;
    return yoco_xattn_decode_status_word(word, wait_class, cta);
}

int32_t yoco_xattn_decode_status_word(int32_t word, int32_t* wait_class, int32_t* cta) {
    if (wait_class) *wait_class = word & 0xFF;
    if (cta) *cta = (int32_t)((uint32_t)word >> 8) - 1;
    return word == kStatusOk ? YOCO_OK : YOCO_ERR_TIMEOUT;
}

int32_t yoco_xattn_selftest_wait_expiry(const yoco_xattn_shape* shape, const void* Q, const void* K, const void* V,
                                        const int32_t* cu_kv_host, const int32_t* kv_len_host, void* O,
                                        void* workspace, size_t workspace_bytes, int32_t limit_ms, void* stream) {
    if (limit_ms <= 0 || limit_ms > 1000) return YOCO_ERR_INVALID_ARG;
    const SelfTest st{(int64_t)limit_ms * 1000000ll};
    return run(shape, YOCO_MODE_DECODE, Q, K, V, cu_kv_host, kv_len_host, O, nullptr, workspace, workspace_bytes,
               stream, nullptr, nullptr, 1, &st);
}

int32_t yoco_xattn_selftest_wait_expiry_fp8(const yoco_xattn_shape* shape, const void* Q, const void* K8,
                                            const void* V8, const float* k_scale_host, const float* v_scale_host,
                                            const int32_t* cu_kv_host, const int32_t* kv_len_host, void* O,
                                            void* workspace, size_t workspace_bytes, int32_t limit_ms, void* stream) {
    if (limit_ms <= 0 || limit_ms > 1000 || !k_scale_host || !v_scale_host) return YOCO_ERR_INVALID_ARG;
    const SelfTest st{(int64_t)limit_ms * 1000000ll};
    const Fp8Scales sc{k_scale_host, v_scale_host};
    return run(shape, YOCO_MODE_DECODE, Q, K8, V8, cu_kv_host, kv_len_host, O, nullptr, workspace, workspace_bytes,
               stream, nullptr, &sc, 1, &st);
}

int32_t yoco_xattn_profile_enable(int32_t max_records) {
    if (max_records < 0) return YOCO_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_mutex);
    for (cudaEvent_t e : g_prof.events) cudaEventDestroy(e);
    g_prof.events.clear();
    g_prof.used = 0;
    for (int32_t k = 0; k < 2 * max_records; ++k) {
        cudaEvent_t e;
        cudaError_t err = cudaEventCreate(&e);
        if (err != cudaSuccess) return cuda_fail(err);
        g_prof.events.push_back(e);
    }
    return YOCO_OK;
}

int32_t yoco_xattn_profile_collect(float* kernel_ms, int32_t capacity, int32_t* count) {
    if (!count || capacity < 0 || (capacity > 0 && !kernel_ms)) return YOCO_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_mutex);
    const int32_t n = std::min(capacity, g_prof.used);
    for (int32_t k = 0; k < n; ++k) {
        YOCO_CUDA_TRY(cudaEventSynchronize(g_prof.events[2 * k + 1]));
        YOCO_CUDA_TRY(cudaEventElapsedTime(&kernel_ms[k], g_prof.events[2 * k], g_prof.events[2 * k + 1]));
    }
    *count = n;
    g_prof.used = 0;
    return YOCO_OK;
}

const char* yoco_xattn_strerror(int32_t code) {
    switch (code) {
        case YOCO_OK: return "ok";
        case YOCO_ERR_INVALID_ARG: return "invalid argument";
        case YOCO_ERR_UNSUPPORTED: return "unsupported shape or device";
        case YOCO_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case YOCO_ERR_CUDA: return "CUDA call failed (see yoco_xattn_last_cuda_error)";
        case YOCO_ERR_TIMEOUT: return "a bounded device-side wait expired";
        case YOCO_ERR_STATIC_SCRATCH_EXCEEDED:
            return "problem needs more scratch than the built-in static buffer holds; "
                   "use yoco_xattn_decode with a caller-provided workspace";
        default: return "unknown error code";
    }
}

int32_t yoco_xattn_last_cuda_error(void) { return g_last_cuda_error; }

}  // extern "C"
