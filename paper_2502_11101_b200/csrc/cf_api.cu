// C ABI entry points: argument checking, buffer layouts, the host-side integer steps.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <mutex>
#include <vector>

#include "cf_common.cuh"

namespace cf {

GeomView make_geom_view(const cf_geom* g) {
    GeomView v;
    v.n_q_heads = g->n_q_heads;
    v.n_kv_heads = g->n_kv_heads;
    v.head_dim = g->head_dim;
    v.dtype = g->dtype;
    v.rope_layout = g->rope_layout;
    v.pos_range = g->pos_range;
    v.rope_theta = g->rope_theta;
    return v;
}

BatchView make_batch_view(const cf_batch* b) {
    BatchView v;
    v.n_requests = b->n_requests;
    v.n_docs_total = b->n_docs_total;
    v.q_len = b->q_len;
    v.prefix_len = b->prefix_len;
    v.tail_reserve = b->tail_reserve;
    v.n_reuse = b->n_reuse;
    v.total_tokens = b->total_tokens;
    v.token_stride = b->token_stride;
    v.req_doc_begin = b->req_doc_begin;
    v.doc_offsets = b->doc_offsets;
    v.doc_src_start = b->doc_src_start;
    return v;
}

int validate(const cf_geom* g, const cf_batch* b) {
    if (!g) return CF_ERR_INVALID_ARG;
    if (g->n_q_heads <= 0 || g->n_kv_heads <= 0 || g->n_q_heads % g->n_kv_heads != 0)
        return CF_ERR_INVALID_ARG;
    if (g->pos_range <= 0 || !(g->rope_theta > 1.0)) return CF_ERR_INVALID_ARG;
    if (g->head_dim != 64 && g->head_dim != 128) return CF_ERR_UNSUPPORTED;
    if (g->dtype != CF_BF16 && g->dtype != CF_F32) return CF_ERR_UNSUPPORTED;
    if (g->rope_layout != CF_ROPE_HALF && g->rope_layout != CF_ROPE_INTERLEAVED)
        return CF_ERR_UNSUPPORTED;
    if (!b) return CF_OK;
    if (b->n_requests <= 0 || b->n_docs_total < 0 || b->q_len <= 0 || b->prefix_len < 0 ||
        b->tail_reserve < 0 || b->n_reuse < 0 || b->tiles_hint < 0 || b->total_tokens < 0)
        return CF_ERR_INVALID_ARG;
    if (b->total_tokens > 0x7fffffffLL - kTile) return CF_ERR_INVALID_ARG;
    if (b->token_stride < (int64_t)g->n_kv_heads * g->head_dim) return CF_ERR_INVALID_ARG;
    // rows are moved in 16-byte vectors
    const int esize = g->dtype == CF_BF16 ? 2 : 4;
    if ((b->token_stride * esize) % 16 != 0) return CF_ERR_INVALID_ARG;
    if (!b->req_doc_begin || !b->doc_offsets || !b->doc_src_start) return CF_ERR_INVALID_ARG;
    if (g->pos_range - b->prefix_len - b->tail_reserve <= 0) return CF_ERR_RANGE;
    return CF_OK;
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static void plan_layout(const cf_geom* g, const cf_batch* b, cf_plan_layout* L) {
    const size_t nd = (size_t)b->n_docs_total, nb = (size_t)b->n_requests;
    const size_t max_tiles = nd + (size_t)(b->total_tokens / kTile) + 1;
    size_t off = 0;
    auto take = [&](size_t count, size_t elem) {
        size_t at = off;
        off = align_up(off + count * elem, 256);
        return at;
    };
    L->status = take(4, 4);
    L->kept = take(nd, 4);
    L->kept_count = take(nb, 4);
    L->dst_start = take(nd, 4);
    L->group = take(nd, 4);
    L->n_reuse = take(nb, 4);
    L->query_start = take(nb, 4);
    L->n_tiles = take(nb, 4);
    L->tile_begin = take(nb, 4);
    L->doc_tile_begin = take(nd, 4);
    L->doc_tile_count = take(nd, 4);
    L->tile_doc = take(max_tiles, 4);
    L->tile_row0 = take(max_tiles, 4);
    L->tile_len = take(max_tiles, 4);
    L->trig = take(nd * (size_t)(g->head_dim / 2), 8);
    L->total_bytes = off;
    L->max_tiles = (int32_t)max_tiles;
    L->reserved = 0;
}

PlanView make_plan_view(const cf_geom* g, const cf_batch* b, void* plan) {
    cf_plan_layout L;
    plan_layout(g, b, &L);
    char* base = static_cast<char*>(plan);
    PlanView v;
    v.status = reinterpret_cast<int*>(base + L.status);
    v.kept = reinterpret_cast<int*>(base + L.kept);
    v.kept_count = reinterpret_cast<int*>(base + L.kept_count);
    v.dst_start = reinterpret_cast<int*>(base + L.dst_start);
    v.group = reinterpret_cast<int*>(base + L.group);
    v.n_reuse = reinterpret_cast<int*>(base + L.n_reuse);
    v.query_start = reinterpret_cast<int*>(base + L.query_start);
    v.n_tiles = reinterpret_cast<int*>(base + L.n_tiles);
    v.tile_begin = reinterpret_cast<int*>(base + L.tile_begin);
    v.doc_tile_begin = reinterpret_cast<int*>(base + L.doc_tile_begin);
    v.doc_tile_count = reinterpret_cast<int*>(base + L.doc_tile_count);
    v.tile_doc = reinterpret_cast<int*>(base + L.tile_doc);
    v.tile_row0 = reinterpret_cast<int*>(base + L.tile_row0);
    v.tile_len = reinterpret_cast<int*>(base + L.tile_len);
    v.trig = reinterpret_cast<float2*>(base + L.trig);
    v.max_tiles = L.max_tiles;
    return v;
}

int current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
    return dev;
}

int sm_count() {
    static std::atomic<int> cached[kMaxDevices] = {};
    const int dev = current_device();
    int n = dev >= 0 ? cached[dev].load() : 0;
    if (n > 0) return n;
    if (dev < 0 || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
        return 148;
    cached[dev].store(n);
    return n;
}

int tiles_per_request_bound(const cf_batch* b) {
    if (b->tiles_hint > 0) return b->tiles_hint;
    long long t = (long long)b->n_docs_total + b->total_tokens / kTile + 1;
    return (int)std::min<long long>(t, 1 << 20);
}

// Query rows one CTA of the tensor-core kernel owns.  A CTA holds two 128-row tiles; when the rows
// that share a kv head fill an odd number of such tiles (and more than one), CTAs of one tile each
// -- whose two warpgroups then take alternate key tiles -- split the work evenly, where pairs would
// leave a half-empty CTA on the critical path.
int choose_row_group(const cf_geom* g, const cf_batch* b) {
    const int rows = (g->n_q_heads / g->n_kv_heads) * b->q_len;
    const int row_tiles = (rows + 127) / 128;
    return (row_tiles > 1 && (row_tiles & 1)) ? 128 : 256;
}

// Parts the key-tile list of a request is cut into.  The tensor-core kernel runs one CTA per
// (layer, request, kv head, group of query rows, pair of parts): as many CTAs as fit one wave over
// the SMs, never more CTAs than tiles.  The count is always even.
int choose_splits(const cf_geom* g, const cf_batch* b, int n_layers) {
    const int rows = (g->n_q_heads / g->n_kv_heads) * b->q_len;
    const int rg_rows = choose_row_group(g, b);
    const int row_groups = (rows + rg_rows - 1) / rg_rows;
    const long long units = (long long)n_layers * b->n_requests * g->n_kv_heads * row_groups;
    const long long sms = sm_count();
    long long s = sms / units;                        // whole CTAs per SM: one wave, no ragged second wave
    if (s == 0) {                                     // more units than SMs: balance the waves instead
        double best = 0.0;
        for (long long c = 1; c <= 4; ++c) {
            const long long ctas = units * c, waves = (ctas + sms - 1) / sms;
            const double eff = (double)ctas / (double)(waves * sms);
            if (eff > best + 0.03) { best = eff; s = c; }
        }
    }
    s = std::min<long long>(s, tiles_per_request_bound(b));
    s = std::min<long long>(s, CF_MAX_SPLITS / 2);
    return 2 * (int)std::max<long long>(s, 1);
}

size_t attn_workspace_layout(const cf_geom* g, const cf_batch* b, int n_splits, int n_layers, bool with_self,
                             AttnWorkspace* ws, void* base_ptr, int part_layers) {
    const size_t rows = (size_t)g->n_q_heads * b->q_len;
    const size_t nlb = (size_t)b->n_requests * (size_t)(part_layers > 0 ? part_layers : n_layers);   // layers of partial results
    const size_t nlb_lse = (size_t)b->n_requests * (size_t)n_layers;
    const size_t max_tiles = (size_t)b->n_docs_total + (size_t)(b->total_tokens / kTile) + 1;
    char* base = static_cast<char*>(base_ptr);
    size_t off = 0;
    auto take = [&](size_t count) {
        size_t at = off;
        off = align_up(off + count * 4, 256);
        return at;
    };
    size_t o = take(nlb * n_splits * rows * g->head_dim);
    size_t m = take(nlb * n_splits * rows);
    size_t l = take(nlb * n_splits * rows);
    size_t t = take((size_t)n_layers * max_tiles * rows);
    size_t r = take(nlb_lse * rows);
    size_t so = 0, sm = 0, sl = 0, ld = 0;
    if (with_self) {                                  // behind everything else: the rest of the layout does not move
        so = take(nlb * rows * g->head_dim);
        sm = take(nlb * rows);
        sl = take(nlb * rows);
        ld = take(nlb * n_splits * rows);
    }
    if (ws) {
        ws->part_o = reinterpret_cast<float*>(base + o);
        ws->part_m = reinterpret_cast<float*>(base + m);
        ws->part_l = reinterpret_cast<float*>(base + l);
        ws->tile_lse2 = reinterpret_cast<float*>(base + t);
        ws->row_lse2 = reinterpret_cast<float*>(base + r);
        ws->n_splits = n_splits;
        ws->part_bf16 = 0;
        ws->n_layers = n_layers;
        ws->max_tiles = (int)max_tiles;
        ws->rg_rows = choose_row_group(g, b);
        ws->self_o = with_self ? reinterpret_cast<float*>(base + so) : nullptr;
        ws->self_m = with_self ? reinterpret_cast<float*>(base + sm) : nullptr;
        ws->self_l = with_self ? reinterpret_cast<float*>(base + sl) : nullptr;
        ws->part_ld = with_self ? reinterpret_cast<float*>(base + ld) : nullptr;
        ws->self_mode = 0;
        ws->keys_in_place = 0;
    }
    return off;
}

static std::atomic<int> g_attn_path{0};
int attn_path() { return g_attn_path.load(); }

// Event pairs around the main attention kernel (cf_profile_begin / cf_profile_end); the three
// variables change together under g_prof_mutex.
static std::mutex g_prof_mutex;
static std::vector<cudaEvent_t> g_prof_events;
static int g_prof_capacity = 0;
static int g_prof_used = 0;

// Claims the next event pair if recording is on; returns its index or -1.
static int prof_claim(cudaEvent_t* start, cudaEvent_t* stop) {
    std::lock_guard<std::mutex> lock(g_prof_mutex);
    if (g_prof_used >= g_prof_capacity) return -1;
    *start = g_prof_events[2 * g_prof_used];
    *stop = g_prof_events[2 * g_prof_used + 1];
    return g_prof_used++;
}

static int check_plan(const cf_geom* geom, const cf_batch* batch, const void* plan) {
    if (!batch || !plan) return CF_ERR_INVALID_ARG;
    int rc = validate(geom, batch);
    if (rc != CF_OK) return rc;
    if (reinterpret_cast<uintptr_t>(plan) % 256 != 0) return CF_ERR_WORKSPACE;
    return CF_OK;
}

int run_attn_layers(const cf_geom* geom, const cf_batch* batch, const void* plan, const LayerSpan& span,
                    const void* q, const void* k_cache, const void* v_cache, const void* k_self,
                    const void* v_self, long long self_stride, float softmax_scale,
                    void* out, float* lse, float* doc_scores, float* score_accum, void* workspace,
                    size_t workspace_bytes, cudaStream_t s, const void* k_prefix, const void* v_prefix,
                    long long prefix_stride, int prefix_len, int slot, int n_slots, bool keys_in_place) {
    int rc = check_plan(geom, batch, plan);
    if (rc != CF_OK) return rc;
    const bool slotted = slot >= 0;                   // one layer into slot `slot` of n_slots, scored later
    if (slotted && (span.n_layers != 1 || n_slots <= 0 || n_slots > CF_MAX_LAYERS_PER_CALL || slot >= n_slots ||
                    doc_scores || score_accum || (long long)n_slots * batch->n_requests > 65535))
        return CF_ERR_INVALID_ARG;
    if (!q || !k_cache || !v_cache || !out || !workspace) return CF_ERR_INVALID_ARG;
    if (!(softmax_scale >= 0.0f) || !std::isfinite(softmax_scale)) return CF_ERR_INVALID_ARG;
    if (span.n_layers <= 0 || span.n_layers > CF_MAX_LAYERS_PER_CALL ||
        (long long)span.n_layers * batch->n_requests > 65535)
        return CF_ERR_INVALID_ARG;
    const int esize = geom->dtype == CF_BF16 ? 2 : 4;
    if (reinterpret_cast<uintptr_t>(workspace) % 256 != 0) return CF_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(q) % 16 || reinterpret_cast<uintptr_t>(out) % 16 ||
        reinterpret_cast<uintptr_t>(k_cache) % 16 || reinterpret_cast<uintptr_t>(v_cache) % 16)
        return CF_ERR_INVALID_ARG;
    if (span.n_layers > 1) {
        const long long layer_rows = (long long)batch->n_requests * batch->q_len * geom->n_q_heads * geom->head_dim;
        if (span.q_stride < layer_rows || span.out_stride < layer_rows ||
            span.kv_stride < batch->total_tokens * batch->token_stride || (span.q_stride * esize) % 16 ||
            (span.out_stride * esize) % 16 || (span.kv_stride * esize) % 16)
            return CF_ERR_INVALID_ARG;
    }
    const bool with_prefix = prefix_len > 0;
    if (with_prefix) {
        const long long layer_rows = (long long)prefix_len * geom->n_kv_heads * geom->head_dim;
        if (!k_prefix || !v_prefix || reinterpret_cast<uintptr_t>(k_prefix) % 16 || reinterpret_cast<uintptr_t>(v_prefix) % 16 ||
            prefix_len > batch->prefix_len || (span.n_layers > 1 && (prefix_stride < layer_rows || (prefix_stride * esize) % 16)))
            return CF_ERR_INVALID_ARG;
    }
    const bool with_self = k_self != nullptr || v_self != nullptr;
    if (with_self) {
        const long long layer_rows = (long long)batch->n_requests * batch->q_len * geom->n_kv_heads * geom->head_dim;
        if (!k_self || !v_self || reinterpret_cast<uintptr_t>(k_self) % 16 || reinterpret_cast<uintptr_t>(v_self) % 16 ||
            (span.n_layers > 1 && (self_stride < layer_rows || (self_stride * esize) % 16)))
            return CF_ERR_INVALID_ARG;
    }
    const int n_splits = choose_splits(geom, batch, span.n_layers);
    AttnWorkspace ws;
    const size_t need = slotted ? attn_workspace_layout(geom, batch, n_splits, n_slots, with_self || with_prefix, &ws, workspace, 1)
                                : attn_workspace_layout(geom, batch, n_splits, span.n_layers, with_self || with_prefix, &ws, workspace);
    if (workspace_bytes < need) return CF_ERR_WORKSPACE;
    if (slotted) {                                    // this call sees its slot as the one layer it has
        const size_t rows_total = (size_t)geom->n_q_heads * batch->q_len;
        ws.tile_lse2 += (size_t)slot * ws.max_tiles * rows_total;
        ws.row_lse2 += (size_t)slot * batch->n_requests * rows_total;
        ws.n_layers = 1;
    }
    const float scale = softmax_scale == 0.0f ? 1.0f / std::sqrt((float)geom->head_dim) : softmax_scale;
    PlanView pv = make_plan_view(geom, batch, const_cast<void*>(plan));
    const bool tensor_core = g_attn_path.load() == 0 && attn_tc_supported(geom, batch);
    if (with_self && batch->q_len > CF_TILE_TOKENS) return CF_ERR_UNSUPPORTED;
    if (!tensor_core) ws.part_ld = nullptr;           // only the tensor-core kernel reports per-part document sums
    if ((with_self || with_prefix) && !tensor_core) { // the CUDA-core path computes these blocks as a part of their own
        ws.self_mode = 1;
        rc = launch_self_block(geom, batch, span, self_stride, q, k_self, v_self, k_prefix, v_prefix, prefix_stride,
                               prefix_len, scale * kLog2e, ws, s);
        if (rc != CF_OK) return rc;
    }
    cudaEvent_t ev_start, ev_stop;
    const bool timed = prof_claim(&ev_start, &ev_stop) >= 0;
    if (timed) cudaEventRecord(ev_start, s);
    ws.keys_in_place = keys_in_place ? 1 : 0;
    if (tensor_core) {
        ws.part_bf16 = 1;
        ws.self_mode = (with_self || with_prefix) ? 2 : 0;   // the blocks ride along as further key tiles
        rc = launch_attn_tc(geom, batch, pv, span, q, k_cache, v_cache, k_self, v_self, self_stride, k_prefix, v_prefix,
                            prefix_stride, prefix_len, scale * kLog2e, ws, s);
    } else
        rc = launch_attn_simt(geom, batch, pv, span, q, k_cache, v_cache, scale * kLog2e, ws, s);
    if (timed) cudaEventRecord(ev_stop, s);
    if (rc != CF_OK) return rc;
    return launch_combine(geom, batch, pv, span, ws, out, lse, doc_scores, score_accum, s);
}

}  // namespace cf

using namespace cf;

extern "C" {

const char* cf_error_string(int code) {
    switch (code) {
        case CF_OK: return "ok";
        case CF_ERR_INVALID_ARG: return "invalid argument";
        case CF_ERR_RANGE: return "kept documents do not fit the positional range";
        case CF_ERR_UNSUPPORTED: return "unsupported geometry";
        case CF_ERR_WORKSPACE: return "plan or workspace buffer too small or misaligned";
        case CF_ERR_CUDA: return "CUDA call failed";
        case CF_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown error";
    }
}

int cf_allocate_positions(const cf_geom* geom, int32_t n_docs, const int32_t* doc_len,
                          const int32_t* order, int32_t n_kept, int32_t prefix_len,
                          int32_t tail_reserve, int32_t n_reuse, int32_t query_start,
                          int32_t* dst_start, int32_t* group, int32_t* n_reuse_out,
                          int32_t* query_start_out) {
    if (!geom || n_docs < 0 || n_kept < 0 || n_kept > n_docs || prefix_len < 0 || tail_reserve < 0 ||
        n_reuse < 0 || !dst_start || !group || (n_docs > 0 && !doc_len) || (n_kept > 0 && !order))
        return CF_ERR_INVALID_ARG;
    const int64_t range = geom->pos_range;
    const int64_t capacity = range - prefix_len - tail_reserve;
    for (int i = 0; i < n_docs; ++i) dst_start[i] = group[i] = -1;
    const int64_t qs = query_start < 0 ? range - tail_reserve : query_start;
    if (n_kept == 0) {
        if (n_reuse_out) *n_reuse_out = std::max(1, n_reuse);
        if (query_start_out) *query_start_out = (int32_t)qs;
        return CF_OK;
    }
    std::vector<char> seen(n_docs, 0);
    int64_t longest = 0;
    for (int r = 0; r < n_kept; ++r) {
        const int i = order[r];
        if (i < 0 || i >= n_docs || seen[i] || doc_len[i] <= 0) return CF_ERR_INVALID_ARG;
        seen[i] = 1;
        longest = std::max<int64_t>(longest, doc_len[i]);
    }
    int64_t windows = n_reuse;
    if (windows <= 0) {
        const int64_t per_window = capacity > 0 ? capacity / longest : 0;   // L / l_C of Eq. 6
        if (per_window <= 0) return CF_ERR_RANGE;
        windows = (n_kept + per_window - 1) / per_window;
    }
    std::vector<int64_t> cursor((size_t)windows, qs);
    for (int r = 0; r < n_kept; ++r) cursor[r % windows] -= doc_len[order[r]];
    if (qs + tail_reserve > range || *std::min_element(cursor.begin(), cursor.end()) < prefix_len)
        return CF_ERR_RANGE;
    std::fill(cursor.begin(), cursor.end(), qs);
    for (int r = 0; r < n_kept; ++r) {
        const int i = order[r];
        const int64_t w = r % windows;
        cursor[w] -= doc_len[i];
        dst_start[i] = (int32_t)cursor[w];
        group[i] = (int32_t)w;
    }
    if (n_reuse_out) *n_reuse_out = (int32_t)windows;
    if (query_start_out) *query_start_out = (int32_t)qs;
    return CF_OK;
}

int cf_schedule_linear(int32_t n_layers, int32_t every, int32_t k, int32_t k_finish,
                       int32_t capacity, int32_t* layers, int32_t* keeps, int32_t* count) {
    if (n_layers <= 0 || every <= 0 || k < 0 || k_finish < 0 || k_finish > k || capacity < 0 || !count)
        return CF_ERR_INVALID_ARG;
    const int prunes = n_layers / every;
    *count = prunes;
    if (prunes == 0) return CF_OK;
    if (capacity < prunes || !layers || !keeps) return CF_ERR_INVALID_ARG;
    const int step = (k - k_finish) / prunes;
    int kept = k;
    for (int j = 1; j <= prunes; ++j) {
        kept = (j == prunes) ? k_finish : kept - step;
        layers[j - 1] = j * every;
        keeps[j - 1] = kept;
    }
    return CF_OK;
}

int cf_plan_layout_of(const cf_geom* geom, const cf_batch* batch, cf_plan_layout* layout) {
    if (!batch || !layout) return CF_ERR_INVALID_ARG;
    int rc = validate(geom, batch);
    if (rc != CF_OK) return rc;
    plan_layout(geom, batch, layout);
    return CF_OK;
}

int cf_plan_init(const cf_geom* geom, const cf_batch* batch, const int32_t* order,
                 const int32_t* kept_count, int32_t query_start, void* plan, size_t plan_bytes,
                 void* stream) {
    int rc = check_plan(geom, batch, plan);
    if (rc != CF_OK) return rc;
    cf_plan_layout L;
    plan_layout(geom, batch, &L);
    if (plan_bytes < L.total_bytes) return CF_ERR_WORKSPACE;
    if (query_start >= 0 && (int64_t)query_start + batch->tail_reserve > geom->pos_range)
        return CF_ERR_RANGE;
    PlanView pv = make_plan_view(geom, batch, plan);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    rc = launch_clear_status(pv, s);
    if (rc != CF_OK) return rc;
    return launch_plan(make_geom_view(geom), make_batch_view(batch), pv, 0, order, kept_count,
                       query_start, nullptr, 0, nullptr, CF_ALLOC_ALIGN, s);
}

int cf_plan_status(const cf_geom* geom, const cf_batch* batch, const void* plan, void* stream) {
    int rc = check_plan(geom, batch, plan);
    if (rc != CF_OK) return rc;
    PlanView pv = make_plan_view(geom, batch, const_cast<void*>(plan));
    int word = 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&word, pv.status, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return CF_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return CF_ERR_CUDA;
    return word;
}

int cf_reposition_keys(const cf_geom* geom, const cf_batch* batch, const void* plan,
                       int32_t n_layers, int64_t layer_stride, const void* k_in, void* k_out,
                       void* stream) {
    int rc = check_plan(geom, batch, plan);
    if (rc != CF_OK) return rc;
    if (!k_in || !k_out || n_layers <= 0) return CF_ERR_INVALID_ARG;
    const int esize = geom->dtype == CF_BF16 ? 2 : 4;
    if (reinterpret_cast<uintptr_t>(k_in) % 16 || reinterpret_cast<uintptr_t>(k_out) % 16 ||
        (layer_stride * esize) % 16)
        return CF_ERR_INVALID_ARG;
    if (n_layers > 1 && layer_stride < batch->total_tokens * batch->token_stride)
        return CF_ERR_INVALID_ARG;
    PlanView pv = make_plan_view(geom, batch, const_cast<void*>(plan));
    return launch_reposition(geom, batch, pv, n_layers, layer_stride, k_in, k_out,
                             static_cast<cudaStream_t>(stream));
}

int cf_merge_attn(const cf_geom* geom, int32_t n_blocks, int32_t q_len, const void* out_a, const float* lse_a,
                  const void* out_b, const float* lse_b, void* out, float* lse, void* stream) {
    int rc = validate(geom, nullptr);
    if (rc != CF_OK) return rc;
    if (n_blocks <= 0 || q_len <= 0 || !out_a || !lse_a || !out_b || !lse_b || !out) return CF_ERR_INVALID_ARG;
    const long long n_rows = (long long)n_blocks * q_len * geom->n_q_heads;
    return launch_merge_attn(geom, n_rows, q_len, out_a, lse_a, out_b, lse_b, out, lse,
                             static_cast<cudaStream_t>(stream));
}

int cf_assemble_final_cache(const cf_geom* geom, const cf_batch* batch, const void* plan,
                            int32_t n_layers, int64_t layer_stride, const void* k_cache, const void* v_cache,
                            int64_t self_layer_stride, const void* k_self, const void* v_self,
                            int32_t out_rows, void* k_out, void* v_out, int32_t* final_rows, void* stream) {
    int rc = check_plan(geom, batch, plan);
    if (rc != CF_OK) return rc;
    if (!k_cache || !v_cache || !k_self || !v_self || !k_out || !v_out || !final_rows || n_layers <= 0 ||
        out_rows <= 0)
        return CF_ERR_INVALID_ARG;
    const int esize = geom->dtype == CF_BF16 ? 2 : 4;
    const void* ptrs[6] = {k_cache, v_cache, k_self, v_self, k_out, v_out};
    for (const void* p : ptrs)
        if (reinterpret_cast<uintptr_t>(p) % 16) return CF_ERR_INVALID_ARG;
    if ((layer_stride * esize) % 16 || (self_layer_stride * esize) % 16) return CF_ERR_INVALID_ARG;
    if (n_layers > 1 && (layer_stride < batch->total_tokens * batch->token_stride ||
                         self_layer_stride < (int64_t)batch->n_requests * batch->q_len * geom->n_kv_heads * geom->head_dim))
        return CF_ERR_INVALID_ARG;
    PlanView pv = make_plan_view(geom, batch, const_cast<void*>(plan));
    return launch_assemble(geom, batch, pv, n_layers, layer_stride, self_layer_stride, out_rows, k_cache, v_cache,
                           k_self, v_self, k_out, v_out, final_rows, static_cast<cudaStream_t>(stream));
}

size_t cf_attn_workspace_bytes_layers(const cf_geom* geom, const cf_batch* batch, int32_t n_layers) {
    if (!batch || validate(geom, batch) != CF_OK || n_layers <= 0 || n_layers > CF_MAX_LAYERS_PER_CALL) return 0;
    return attn_workspace_layout(geom, batch, choose_splits(geom, batch, n_layers), n_layers, false, nullptr, nullptr);
}

size_t cf_attn_workspace_bytes_full(const cf_geom* geom, const cf_batch* batch, int32_t n_layers) {
    if (!batch || validate(geom, batch) != CF_OK || n_layers <= 0 || n_layers > CF_MAX_LAYERS_PER_CALL) return 0;
    return attn_workspace_layout(geom, batch, choose_splits(geom, batch, n_layers), n_layers, true, nullptr, nullptr);
}

size_t cf_attn_workspace_bytes(const cf_geom* geom, const cf_batch* batch) {
    return cf_attn_workspace_bytes_layers(geom, batch, 1);
}

int cf_profile_begin(int32_t max_records) {
    std::lock_guard<std::mutex> lock(g_prof_mutex);
    if (max_records <= 0 || max_records > (1 << 20) || g_prof_capacity != 0) return CF_ERR_INVALID_ARG;
    g_prof_events.resize(2 * (size_t)max_records);
    for (auto& e : g_prof_events)
        if (cudaEventCreate(&e) != cudaSuccess) return CF_ERR_CUDA;
    g_prof_used = 0;
    g_prof_capacity = max_records;
    return CF_OK;
}

int cf_profile_end(float* ms, int32_t capacity, int32_t* count) {
    if (!count || capacity < 0 || (capacity > 0 && !ms)) return CF_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_prof_mutex);
    int rc = CF_OK;
    const int n = g_prof_used;
    for (int i = 0; i < n; ++i) {
        float t = 0.f;
        if (cudaEventSynchronize(g_prof_events[2 * i + 1]) != cudaSuccess ||
            cudaEventElapsedTime(&t, g_prof_events[2 * i], g_prof_events[2 * i + 1]) != cudaSuccess)
            rc = CF_ERR_CUDA;
        if (i < capacity) ms[i] = t;
    }
    for (auto& e : g_prof_events) cudaEventDestroy(e);
    g_prof_events.clear();
    g_prof_capacity = g_prof_used = 0;
    *count = n;
    return rc;
}

int cf_set_attn_path(int32_t path) {
    if (path != 0 && path != 1) return CF_ERR_INVALID_ARG;
    g_attn_path.store(path);
    return CF_OK;
}

int cf_query_prefill_attn(const cf_geom* geom, const cf_batch* batch, const void* plan,
                          const void* q, const void* k_cache, const void* v_cache,
                          float softmax_scale, void* out, float* lse, float* doc_scores,
                          float* score_accum, void* workspace, size_t workspace_bytes,
                          void* stream) {
    const LayerSpan span = {1, 0, 0, 0};
    return run_attn_layers(geom, batch, plan, span, q, k_cache, v_cache, nullptr, nullptr, 0, softmax_scale, out, lse,
                           doc_scores, score_accum, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

int cf_query_prefill_attn_layers(const cf_geom* geom, const cf_batch* batch, const void* plan,
                                 int32_t n_layers, const void* q, int64_t q_layer_stride,
                                 const void* k_cache, const void* v_cache, int64_t kv_layer_stride,
                                 float softmax_scale, void* out, int64_t out_layer_stride,
                                 float* lse, float* doc_scores, float* score_accum,
                                 void* workspace, size_t workspace_bytes, void* stream) {
    if (q_layer_stride < 0 || kv_layer_stride < 0 || out_layer_stride < 0) return CF_ERR_INVALID_ARG;
    const LayerSpan span = {n_layers, q_layer_stride, kv_layer_stride, out_layer_stride};
    return run_attn_layers(geom, batch, plan, span, q, k_cache, v_cache, nullptr, nullptr, 0, softmax_scale, out, lse,
                           doc_scores, score_accum, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

size_t cf_attn_workspace_bytes_slots(const cf_geom* geom, const cf_batch* batch, int32_t n_slots) {
    if (!batch || validate(geom, batch) != CF_OK || n_slots <= 0 || n_slots > CF_MAX_LAYERS_PER_CALL) return 0;
    return attn_workspace_layout(geom, batch, choose_splits(geom, batch, 1), n_slots, false, nullptr, nullptr, 1);
}

int cf_query_prefill_attn_slot(const cf_geom* geom, const cf_batch* batch, const void* plan, int32_t slot,
                               int32_t n_slots, const void* q, const void* k_cache, const void* v_cache,
                               float softmax_scale, void* out, float* lse, void* workspace, size_t workspace_bytes,
                               void* stream) {
    if (slot < 0) return CF_ERR_INVALID_ARG;
    const LayerSpan span = {1, 0, 0, 0};
    return run_attn_layers(geom, batch, plan, span, q, k_cache, v_cache, nullptr, nullptr, 0, softmax_scale, out, lse,
                           nullptr, nullptr, workspace, workspace_bytes, static_cast<cudaStream_t>(stream), nullptr, nullptr,
                           0, 0, slot, n_slots);
}

size_t cf_attn_workspace_bytes_slots_full(const cf_geom* geom, const cf_batch* batch, int32_t n_slots) {
    if (!batch || validate(geom, batch) != CF_OK || n_slots <= 0 || n_slots > CF_MAX_LAYERS_PER_CALL) return 0;
    return attn_workspace_layout(geom, batch, choose_splits(geom, batch, 1), n_slots, true, nullptr, nullptr, 1);
}

int cf_query_prefill_attn_slot_full(const cf_geom* geom, const cf_batch* batch, const void* plan, int32_t slot,
                                    int32_t n_slots, const void* q, const void* k_cache, const void* v_cache,
                                    const void* k_prefix, const void* v_prefix, int32_t prefix_len, const void* k_self,
                                    const void* v_self, float softmax_scale, void* out, float* lse, void* workspace,
                                    size_t workspace_bytes, void* stream) {
    if (slot < 0 || prefix_len < 0 || (prefix_len == 0 && !k_self) || (k_self == nullptr) != (v_self == nullptr))
        return CF_ERR_INVALID_ARG;
    const LayerSpan span = {1, 0, 0, 0};
    return run_attn_layers(geom, batch, plan, span, q, k_cache, v_cache, k_self, v_self, 0, softmax_scale, out, lse,
                           nullptr, nullptr, workspace, workspace_bytes, static_cast<cudaStream_t>(stream),
                           prefix_len > 0 ? k_prefix : nullptr, prefix_len > 0 ? v_prefix : nullptr, 0, prefix_len, slot,
                           n_slots);
}

int cf_accumulate_scores(const cf_geom* geom, const cf_batch* batch, const void* plan, int32_t n_filled, int32_t n_slots,
                         float* doc_scores, float* score_accum, void* workspace, size_t workspace_bytes, void* stream) {
    int rc = check_plan(geom, batch, plan);
    if (rc != CF_OK) return rc;
    if (n_slots <= 0 || n_slots > CF_MAX_LAYERS_PER_CALL || n_filled <= 0 || n_filled > n_slots || !workspace)
        return CF_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) % 256 != 0) return CF_ERR_WORKSPACE;
    AttnWorkspace ws;
    const size_t need = attn_workspace_layout(geom, batch, choose_splits(geom, batch, 1), n_slots, false, &ws, workspace, 1);
    if (workspace_bytes < need) return CF_ERR_WORKSPACE;
    ws.n_layers = n_filled;
    return launch_scores(geom, batch, make_plan_view(geom, batch, const_cast<void*>(plan)), ws, doc_scores, score_accum,
                         static_cast<cudaStream_t>(stream));
}

int cf_query_prefill_attn_full(const cf_geom* geom, const cf_batch* batch, const void* plan,
                               int32_t n_layers, const void* q, int64_t q_layer_stride,
                               const void* k_cache, const void* v_cache, int64_t kv_layer_stride,
                               const void* k_self, const void* v_self, int64_t self_layer_stride,
                               float softmax_scale, void* out, int64_t out_layer_stride,
                               float* lse, float* doc_scores, float* score_accum,
                               void* workspace, size_t workspace_bytes, void* stream) {
    if (q_layer_stride < 0 || kv_layer_stride < 0 || out_layer_stride < 0 || self_layer_stride < 0 || !k_self || !v_self)
        return CF_ERR_INVALID_ARG;
    const LayerSpan span = {n_layers, q_layer_stride, kv_layer_stride, out_layer_stride};
    return run_attn_layers(geom, batch, plan, span, q, k_cache, v_cache, k_self, v_self, self_layer_stride,
                           softmax_scale, out, lse, doc_scores, score_accum, workspace, workspace_bytes,
                           static_cast<cudaStream_t>(stream));
}

int cf_query_prefill_attn_prefix(const cf_geom* geom, const cf_batch* batch, const void* plan,
                                 int32_t n_layers, const void* q, int64_t q_layer_stride,
                                 const void* k_cache, const void* v_cache, int64_t kv_layer_stride,
                                 const void* k_prefix, const void* v_prefix, int64_t prefix_layer_stride,
                                 int32_t prefix_len, const void* k_self, const void* v_self,
                                 int64_t self_layer_stride, float softmax_scale, void* out,
                                 int64_t out_layer_stride, float* lse, float* doc_scores, float* score_accum,
                                 void* workspace, size_t workspace_bytes, void* stream) {
    if (q_layer_stride < 0 || kv_layer_stride < 0 || out_layer_stride < 0 || self_layer_stride < 0 ||
        prefix_layer_stride < 0 || prefix_len <= 0 || !k_prefix || !v_prefix || (k_self == nullptr) != (v_self == nullptr))
        return CF_ERR_INVALID_ARG;
    const LayerSpan span = {n_layers, q_layer_stride, kv_layer_stride, out_layer_stride};
    return run_attn_layers(geom, batch, plan, span, q, k_cache, v_cache, k_self, v_self, self_layer_stride,
                           softmax_scale, out, lse, doc_scores, score_accum, workspace, workspace_bytes,
                           static_cast<cudaStream_t>(stream), k_prefix, v_prefix, prefix_layer_stride, prefix_len);
}

int cf_prune_topk(const cf_geom* geom, const cf_batch* batch, void* plan,
                  const float* score_accum, int32_t keep, const int32_t* keep_per_request,
                  int32_t strategy, void* stream) {
    int rc = check_plan(geom, batch, plan);
    if (rc != CF_OK) return rc;
    if (!score_accum || (keep < 0 && !keep_per_request)) return CF_ERR_INVALID_ARG;
    if (strategy != CF_ALLOC_NONE && strategy != CF_ALLOC_ALIGN && strategy != CF_ALLOC_SORT)
        return CF_ERR_INVALID_ARG;
    PlanView pv = make_plan_view(geom, batch, plan);
    return launch_plan(make_geom_view(geom), make_batch_view(batch), pv, 1, nullptr, nullptr, -1,
                       score_accum, keep, keep_per_request, strategy,
                       static_cast<cudaStream_t>(stream));
}

}  // extern "C"
