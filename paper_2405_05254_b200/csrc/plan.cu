// Split-count / tile planner: pure host integer code, deterministic.
#include "plan.h"

#include <algorithm>
#include <climits>

namespace yoco {

int32_t validate_shape(const yoco_xattn_shape& s, int32_t mode) {
    if (s.B < 0 || s.Hq <= 0 || s.Hkv <= 0 || s.T <= 0 || s.d <= 0 || s.max_kv_len < 0 ||
        s.kv_head_stride < 0 || s.window < 0 || !(s.scale >= 0.f))
        return YOCO_ERR_INVALID_ARG;
    if (mode != YOCO_MODE_DECODE && mode != YOCO_MODE_CHUNK) return YOCO_ERR_INVALID_ARG;
    if (s.d != 64 && s.d != 128) return YOCO_ERR_UNSUPPORTED;
    if (s.Hq % s.Hkv != 0) return YOCO_ERR_UNSUPPORTED;
    if (s.kv_head_stride % s.d != 0) return YOCO_ERR_UNSUPPORTED;
    const int64_t rows = (int64_t)(s.Hq / s.Hkv) * s.T;
    if (mode == YOCO_MODE_DECODE && rows > kDecodeTileM) return YOCO_ERR_UNSUPPORTED;
    if ((int64_t)s.B * s.Hq * s.T >= (1ll << 31)) return YOCO_ERR_UNSUPPORTED;
    return YOCO_OK;
}

int32_t validate_layout(const yoco_xattn_shape& s, const int32_t* cu_kv_host, const int32_t* kv_len_host) {
    for (int i = 0; i < s.B; ++i) {
        const int64_t n = kv_len_host ? kv_len_host[i] : s.max_kv_len;
        if (n < 0) return YOCO_ERR_INVALID_ARG;
        const int64_t head_rows = s.kv_head_stride ? s.kv_head_stride / s.d : n;
        if (head_rows < n) return YOCO_ERR_INVALID_ARG;
        if (cu_kv_host) {
            if (cu_kv_host[i] < 0 || cu_kv_host[i + 1] < cu_kv_host[i]) return YOCO_ERR_INVALID_ARG;
            // sequence i occupies Hkv * head_rows rows from token offset cu[i]: the next one may not start inside it
            if (n > 0 && (int64_t)cu_kv_host[i + 1] - cu_kv_host[i] < head_rows) return YOCO_ERR_INVALID_ARG;
        }
    }
    return YOCO_OK;
}

int32_t make_plan(const yoco_xattn_shape& s, const int32_t* cu_kv_host, const int32_t* kv_len_host,
                  int32_t sm_count, int32_t mode, Plan& plan, int32_t max_sub_items,
                  const int32_t* key_offset_host, const int32_t* kv_total_host, bool eight_bit_cache) {
    int32_t rc = validate_shape(s, mode);
    if (rc != YOCO_OK) return rc;
    if (sm_count <= 0) return YOCO_ERR_INVALID_ARG;
    if ((rc = validate_layout(s, cu_kv_host, kv_len_host)) != YOCO_OK) return rc;

    const int G = s.Hq / s.Hkv;
    const int rows_per_stream = G * s.T;
    const int tile_n = mode == YOCO_MODE_DECODE ? kDecodeTileN : kChunkTileN;
    const int tile_m = mode == YOCO_MODE_DECODE ? kDecodeTileM
                       : (rows_per_stream > kChunkTileM || eight_bit_cache) ? kChunkPairTileM : kChunkTileM;
    const int m_tiles = (rows_per_stream + tile_m - 1) / tile_m;
    const int num_streams = s.B * s.Hkv;

    // per-sequence geometry
    if ((key_offset_host == nullptr) != (kv_total_host == nullptr)) return YOCO_ERR_INVALID_ARG;
    std::vector<int64_t> tok_off(s.B + 1, 0);
    std::vector<int32_t> len(s.B, 0);
    std::vector<int64_t> n_full(s.B, 0);     // keys of this cache that query row 0 sees (see DevSegment)
    std::vector<int32_t> len_vis(s.B, 0);    // keys of this cache that at least the last row sees
    int64_t extent = 0;
    for (int i = 0; i < s.B; ++i) {
        len[i] = kv_len_host ? kv_len_host[i] : s.max_kv_len;
        if (key_offset_host) {
            if (key_offset_host[i] < 0 || len[i] < 0 || (int64_t)key_offset_host[i] + len[i] > kv_total_host[i])
                return YOCO_ERR_INVALID_ARG;
            n_full[i] = (int64_t)kv_total_host[i] - s.T + 1 - key_offset_host[i];
        } else {
            n_full[i] = (int64_t)len[i] - s.T + 1;
        }
        len_vis[i] = (int32_t)std::min<int64_t>(std::max<int64_t>(len[i], 0), std::max<int64_t>(n_full[i] + s.T - 1, 0));
        if (cu_kv_host) tok_off[i] = cu_kv_host[i];
        const int64_t head_rows = s.kv_head_stride ? s.kv_head_stride / s.d : len[i];
        if (!cu_kv_host) tok_off[i + 1] = tok_off[i] + head_rows;
        if (len[i] > 0)
            extent = std::max(extent, tok_off[i] * s.Hkv + (int64_t)(s.Hkv - 1) * head_rows + len[i]);
    }
    if (extent >= (1ll << 31)) return YOCO_ERR_UNSUPPORTED;

    // With a sliding window the lowest key any row of the call sees is that of row 0:
    // (N - T) - C + 1.  Whole tiles below it are left out of the plan.
    std::vector<int64_t> tile_lo(s.B, 0);
    int64_t total_tiles = 0;
    for (int i = 0; i < s.B; ++i) {
        if (s.window > 0) {
            const int64_t lo = n_full[i] - s.window;      // lowest key row 0 sees
            tile_lo[i] = std::min<int64_t>(std::max<int64_t>(lo, 0) / tile_n, (len_vis[i] + tile_n - 1) / tile_n);
        }
        total_tiles += (int64_t)s.Hkv * ((len_vis[i] + tile_n - 1) / tile_n - tile_lo[i]);
    }

    // number of CTA groups
    int64_t target;
    if (mode == YOCO_MODE_DECODE)
        target = (int64_t)sm_count * kDecodeGroupsPerSm;
    else
        target = std::max<int64_t>(1, sm_count / m_tiles);
    const int64_t num_groups = std::max<int64_t>(1, std::min<int64_t>(target, total_tiles));

    plan = Plan{};
    plan.rows_per_stream = rows_per_stream;
    plan.kv_rows_extent = extent;
    std::vector<int32_t> group_begin(num_groups + 1, 0);
    std::vector<int32_t> stream_base(num_streams, 0), stream_nseg(num_streams, 0);
    std::vector<DevSegment> dev;

    // walk the flat tile space: streams in (b, c) order
    int64_t flat = 0;       // flat index of the current stream's first tile
    int64_t g = 0;          // current group
    auto group_lo = [&](int64_t p) { return p * total_tiles / num_groups; };
    for (int b = 0; b < s.B; ++b) {
        const int64_t nt = (len_vis[b] + tile_n - 1) / tile_n;
        const int64_t head_rows = s.kv_head_stride ? s.kv_head_stride / s.d : len[b];
        for (int c = 0; c < s.Hkv; ++c) {
            const int stream = b * s.Hkv + c;
            stream_base[stream] = (int32_t)dev.size();
            const int64_t t0 = tile_lo[b];
            int64_t t = t0;  // tile inside the stream
            while (t < nt) {
                while (group_lo(g + 1) <= flat + (t - t0)) ++g;     // group owning this flat tile
                const int64_t t_end = std::min<int64_t>(nt, group_lo(g + 1) - flat + t0);
                DevSegment d{};
                d.k_begin = (int32_t)(t * tile_n);
                d.k_end = (int32_t)std::min<int64_t>(t_end * tile_n, len_vis[b]);
                d.kv_row0 = (int32_t)(tok_off[b] * s.Hkv + c * head_rows + d.k_begin);
                d.q_row0 = (b * s.Hq + c * G) * s.T;
                d.slot = (int32_t)dev.size();
                d.n_kv = len[b];
                d.stream = stream;
                d.n_full = (int32_t)std::max<int64_t>(std::min<int64_t>(n_full[b], INT32_MAX), INT32_MIN / 2);
                yoco_xattn_segment pub{(int32_t)g, b, c, d.k_begin, d.k_end, d.slot};
                plan.segments.push_back(pub);
                dev.push_back(d);
                ++stream_nseg[stream];
                t = t_end;
            }
            flat += nt - t0;
        }
    }
    // Pieces pay when a group is one long run of a stream.  When groups are chains of short streams
    // (more than two segments per group on average) most streams are not split at all and are written
    // without a merge; pieces would split every one of them.
    int R = mode == YOCO_MODE_DECODE ? choose_sub_items(total_tiles / num_groups / (eight_bit_cache ? 2 : 1), max_sub_items) : 1;
    if ((int64_t)dev.size() > 2 * num_groups) R = 1;
    int32_t max_splits = 0, needs_combine = R > 1 ? 1 : 0;
    for (int st = 0; st < num_streams; ++st) {
        max_splits = std::max(max_splits, stream_nseg[st] * R);
        if (stream_nseg[st] != 1) needs_combine = 1;
    }
    for (auto& d : dev) d.stream_nseg = stream_nseg[d.stream];
    // group offsets (segments are already sorted by group)
    {
        size_t k = 0;
        for (int64_t p = 0; p < num_groups; ++p) {
            group_begin[p] = (int32_t)k;
            while (k < plan.segments.size() && plan.segments[k].group == p) ++k;
        }
        group_begin[num_groups] = (int32_t)k;
    }

    // With R > 1 the public list names the pieces that are executed: piece r of group g is work
    // item r * num_groups + g and fills slot (segment index) * R + r.  Same walk as the kernel's.
    if (R > 1) {
        std::vector<yoco_xattn_segment> pieces;
        for (int64_t p = 0; p < num_groups; ++p) {
            int64_t n_g = 0;
            for (int32_t k = group_begin[p]; k < group_begin[p + 1]; ++k)
                n_g += (dev[k].k_end - dev[k].k_begin + tile_n - 1) / tile_n;
            int64_t acc = 0;
            for (int32_t k = group_begin[p]; k < group_begin[p + 1]; ++k) {
                const int64_t nt = (dev[k].k_end - dev[k].k_begin + tile_n - 1) / tile_n;
                for (int r = 0; r < R; ++r) {
                    const int64_t lo = std::max<int64_t>(sub_bound(n_g, R, r) - acc, 0);
                    const int64_t hi = std::min<int64_t>(sub_bound(n_g, R, r + 1) - acc, nt);
                    if (lo >= hi) continue;
                    yoco_xattn_segment pub = plan.segments[k];
                    pub.group = (int32_t)(r * num_groups + p);
                    pub.k_begin = (int32_t)(dev[k].k_begin + lo * tile_n);
                    pub.k_end = (int32_t)std::min<int64_t>(dev[k].k_begin + hi * tile_n, dev[k].k_end);
                    pub.slot = dev[k].slot * R + r;
                    pieces.push_back(pub);
                }
                acc += nt;
            }
        }
        plan.segments.swap(pieces);
    }
    plan.sub_items = R;
    plan.coarse_segments = (int32_t)dev.size();

    // device blob
    plan.off_segments = 0;
    plan.off_group_begin = (int32_t)(dev.size() * kSegmentWords);
    plan.off_stream_base = plan.off_group_begin + (int32_t)group_begin.size();
    plan.off_stream_nseg = plan.off_stream_base + num_streams;
    plan.table.resize(plan.off_stream_nseg + num_streams);
    static_assert(sizeof(DevSegment) == 4 * kSegmentWords, "DevSegment is kSegmentWords int32");
    for (size_t k = 0; k < dev.size(); ++k) {
        const int32_t* w = reinterpret_cast<const int32_t*>(&dev[k]);
        std::copy(w, w + kSegmentWords, plan.table.begin() + k * kSegmentWords);
    }
    std::copy(group_begin.begin(), group_begin.end(), plan.table.begin() + plan.off_group_begin);
    std::copy(stream_base.begin(), stream_base.end(), plan.table.begin() + plan.off_stream_base);
    std::copy(stream_nseg.begin(), stream_nseg.end(), plan.table.begin() + plan.off_stream_nseg);

    auto align256 = [](int64_t x) { return (x + 255) / 256 * 256; };
    plan.ws_table = kWorkspaceHeaderBytes;
    plan.ws_part_lse = align256(plan.ws_table + (int64_t)plan.table.size() * 4);
    const int64_t slots = (int64_t)dev.size() * R;
    plan.ws_part_o = align256(plan.ws_part_lse + slots * rows_per_stream * 4);
    const int64_t ws_end = align256(plan.ws_part_o + slots * rows_per_stream * s.d * 4);

    yoco_xattn_plan_info& info = plan.info;
    info.mode = mode;
    info.tile_n = tile_n;
    info.tile_m = tile_m;
    info.m_tiles = m_tiles;
    info.num_groups = (int32_t)num_groups;
    info.num_ctas = (int32_t)(num_groups * m_tiles);
    info.num_streams = num_streams;
    info.num_segments = (int32_t)plan.segments.size();
    info.sub_items = R;
    info.num_slots = (int32_t)slots;
    info.max_splits = max_splits;
    info.needs_combine = needs_combine;
    info.total_tiles = total_tiles;
    info.workspace_bytes = ws_end;
    return YOCO_OK;
}

}  // namespace yoco
