// Algorithm 2, Phases 1 and 2, sequenced by the library itself (cf_run_stack), the host-side mirror of
// the pruning step (cf_prune_topk_host), and the probe of the bounded device-side wait.
#include <algorithm>
#include <cmath>
#include <vector>

#include "cf_common.cuh"

namespace cf {

namespace {

// Layers [first, last) that go to the library's attention in one call.
struct Call {
    int first, last;
    int prune_after;       // index into the schedule of the pruning step that follows the call, -1 if none
};

bool schedule_ok(const cf_stack* st) {
    if (st->n_prune < 0 || (st->n_prune > 0 && (!st->prune_layer || !st->prune_keep))) return false;
    int prev = 0;
    for (int i = 0; i < st->n_prune; ++i) {
        if (st->prune_layer[i] <= prev || st->prune_keep[i] < 0) return false;   // 1-based, strictly ascending
        prev = st->prune_layer[i];
    }
    return true;
}

// The attention calls of a stack.  Pruning layers beyond the last layer never fire (Algorithm 2 tests
// `l mod n = 0` inside the loop over layers).
std::vector<Call> calls_of(const cf_stack* st) {
    std::vector<Call> calls;
    const int n = st->n_layers;
    if (!st->batch_layers) {
        int next = 0;
        for (int l = 1; l <= n; ++l) {
            int after = -1;
            if (next < st->n_prune && st->prune_layer[next] == l) after = next++;
            calls.push_back({l - 1, l, after});
        }
        return calls;
    }
    int first = 0;
    for (int i = 0; i <= st->n_prune; ++i) {
        const bool is_cut = i < st->n_prune && st->prune_layer[i] <= n;
        const int last = is_cut ? st->prune_layer[i] : n;
        for (int lo = first; lo < last; lo += CF_MAX_LAYERS_PER_CALL) {
            const int hi = std::min(last, lo + CF_MAX_LAYERS_PER_CALL);
            calls.push_back({lo, hi, (is_cut && hi == last) ? i : -1});
        }
        if (!is_cut) break;
        first = last;
    }
    return calls;
}

// Upper bound of the key tiles a request can own while it keeps at most `keep` documents: the tile
// counts of its `keep` longest documents (only steers grid sizes).  0 when the lengths are unknown.
int live_tiles_hint(const cf_batch* b, const cf_stack* st, int keep) {
    if (!st->doc_len_host || !st->req_doc_begin_host) return b->tiles_hint;
    int worst = 1;
    std::vector<int> tiles;
    for (int r = 0; r < b->n_requests; ++r) {
        const int lo = st->req_doc_begin_host[r], hi = st->req_doc_begin_host[r + 1];
        tiles.clear();
        for (int i = lo; i < hi; ++i) tiles.push_back((st->doc_len_host[i] + kTile - 1) / kTile);
        std::sort(tiles.begin(), tiles.end(), std::greater<int>());
        int sum = 0;
        for (int i = 0; i < (int)tiles.size() && i < keep; ++i) sum += tiles[i];
        worst = std::max(worst, sum);
    }
    return worst;
}

int max_docs_per_request(const cf_batch* b, const cf_stack* st) {
    if (!st->req_doc_begin_host) return b->n_docs_total;
    int worst = 0;
    for (int r = 0; r < b->n_requests; ++r)
        worst = std::max(worst, st->req_doc_begin_host[r + 1] - st->req_doc_begin_host[r]);
    return worst;
}

// With one attention call per layer the layers' document scores are
// left in slots of the workspace and added to S together: right before a pruning layer uses S, when the
// slots are full, and after the last layer (cf_query_prefill_attn_slot, cf_accumulate_scores).
constexpr int kScoreSlots = 8;
bool deferred_scores(const cf_stack* st) { return !st->batch_layers; }
int score_slots(const cf_stack* st) { return std::min(kScoreSlots, st->n_layers); }

int check_stack(const cf_geom* geom, const cf_batch* batch, const cf_stack* st) {
    if (!batch || !st) return CF_ERR_INVALID_ARG;
    int rc = validate(geom, batch);
    if (rc != CF_OK) return rc;
    if (st->n_layers <= 0 || !schedule_ok(st)) return CF_ERR_INVALID_ARG;
    if (st->strategy != CF_ALLOC_NONE && st->strategy != CF_ALLOC_ALIGN && st->strategy != CF_ALLOC_SORT)
        return CF_ERR_INVALID_ARG;
    if ((st->k_self == nullptr) != (st->v_self == nullptr)) return CF_ERR_INVALID_ARG;
    if (st->prefix_len < 0 || (st->prefix_len > 0 && (!st->k_prefix || !st->v_prefix))) return CF_ERR_INVALID_ARG;
    return CF_OK;
}

}  // namespace

}  // namespace cf

using namespace cf;

extern "C" {

size_t cf_run_stack_workspace_bytes(const cf_geom* geom, const cf_batch* batch, const cf_stack* stack) {
    if (check_stack(geom, batch, stack) != CF_OK) return 0;
    cf_batch local = *batch;
    int keep = max_docs_per_request(batch, stack);
    size_t need = 0;
    for (const Call& c : calls_of(stack)) {
        local.tiles_hint = live_tiles_hint(batch, stack, keep);
        const int m = c.last - c.first;
        const bool blocks = stack->k_self || stack->prefix_len > 0;
        need = std::max(need, deferred_scores(stack)
                                  ? (blocks ? cf_attn_workspace_bytes_slots_full(geom, &local, score_slots(stack))
                                            : cf_attn_workspace_bytes_slots(geom, &local, score_slots(stack)))
                                  : (blocks ? cf_attn_workspace_bytes_full(geom, &local, m)
                                            : cf_attn_workspace_bytes_layers(geom, &local, m)));
        if (c.prune_after >= 0) keep = std::min(keep, stack->prune_keep[c.prune_after]);
    }
    return need;
}

int cf_run_stack(const cf_geom* geom, const cf_batch* batch, const cf_stack* stack, void* plan, size_t plan_bytes,
                 void* workspace, size_t workspace_bytes, void* stream) {
    int rc = check_stack(geom, batch, stack);
    if (rc != CF_OK) return rc;
    if (!stack->q || !stack->k_cache || !stack->v_cache || !stack->out || !stack->score_accum || !plan || !workspace)
        return CF_ERR_INVALID_ARG;
    if (stack->n_layers > 1 && (stack->q_layer_stride <= 0 || stack->kv_layer_stride <= 0 || stack->out_layer_stride <= 0 ||
                                (stack->k_self && stack->self_layer_stride <= 0) ||
                                (stack->prefix_len > 0 && stack->prefix_layer_stride <= 0)))
        return CF_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t esize = geom->dtype == CF_BF16 ? 2 : 4;
    const size_t nd = (size_t)batch->n_docs_total;
    const size_t lse_layer = (size_t)batch->n_requests * geom->n_q_heads * batch->q_len;

    // Init: S = 0, every document kept in retrieval order, first allocation
    if (nd > 0 && cudaMemsetAsync(stack->score_accum, 0, nd * sizeof(float), s) != cudaSuccess) return CF_ERR_CUDA;
    cf_batch local = *batch;
    int keep = max_docs_per_request(batch, stack);
    local.tiles_hint = live_tiles_hint(batch, stack, keep);
    rc = cf_plan_init(geom, &local, nullptr, nullptr, -1, plan, plan_bytes, stream);
    if (rc != CF_OK) return rc;

    // Phase 1: layer_l (attention over the kept caches, S += s^l), pruning and re-allocation at the scheduled layers
    const bool deferred = deferred_scores(stack);
    const int n_slots = score_slots(stack);
    int filled = 0;                                                 // layers whose scores wait in the workspace
    for (const Call& c : calls_of(stack)) {
        const int m = c.last - c.first;
        const char* q = static_cast<const char*>(stack->q) + (size_t)c.first * stack->q_layer_stride * esize;
        const char* k = static_cast<const char*>(stack->k_cache) + (size_t)c.first * stack->kv_layer_stride * esize;
        const char* v = static_cast<const char*>(stack->v_cache) + (size_t)c.first * stack->kv_layer_stride * esize;
        char* out = static_cast<char*>(stack->out) + (size_t)c.first * stack->out_layer_stride * esize;
        float* lse = stack->lse ? stack->lse + (size_t)c.first * lse_layer : nullptr;
        float* scores = stack->layer_scores ? stack->layer_scores + (size_t)c.first * nd : nullptr;
        if (deferred) {
            const char* ks = stack->k_self ? static_cast<const char*>(stack->k_self) + (size_t)c.first * stack->self_layer_stride * esize : nullptr;
            const char* vs = stack->v_self ? static_cast<const char*>(stack->v_self) + (size_t)c.first * stack->self_layer_stride * esize : nullptr;
            const char* kp = stack->prefix_len > 0 ? static_cast<const char*>(stack->k_prefix) + (size_t)c.first * stack->prefix_layer_stride * esize : nullptr;
            const char* vp = stack->prefix_len > 0 ? static_cast<const char*>(stack->v_prefix) + (size_t)c.first * stack->prefix_layer_stride * esize : nullptr;
            rc = (ks || kp) ? cf_query_prefill_attn_slot_full(geom, &local, plan, filled, n_slots, q, k, v, kp, vp,
                                                              stack->prefix_len, ks, vs, stack->softmax_scale, out, lse,
                                                              workspace, workspace_bytes, stream)
                            : cf_query_prefill_attn_slot(geom, &local, plan, filled, n_slots, q, k, v, stack->softmax_scale,
                                                         out, lse, workspace, workspace_bytes, stream);
            if (rc != CF_OK) return rc;
            ++filled;
            if (c.prune_after >= 0 || filled == n_slots || c.last == stack->n_layers) {
                float* first = stack->layer_scores ? stack->layer_scores + (size_t)(c.last - filled) * nd : nullptr;
                rc = cf_accumulate_scores(geom, &local, plan, filled, n_slots, first, stack->score_accum, workspace,
                                          workspace_bytes, stream);
                filled = 0;
            }
        } else if (stack->prefix_len > 0) {
            const char* ks = stack->k_self ? static_cast<const char*>(stack->k_self) + (size_t)c.first * stack->self_layer_stride * esize : nullptr;
            const char* vs = stack->v_self ? static_cast<const char*>(stack->v_self) + (size_t)c.first * stack->self_layer_stride * esize : nullptr;
            const char* kp = static_cast<const char*>(stack->k_prefix) + (size_t)c.first * stack->prefix_layer_stride * esize;
            const char* vp = static_cast<const char*>(stack->v_prefix) + (size_t)c.first * stack->prefix_layer_stride * esize;
            rc = cf_query_prefill_attn_prefix(geom, &local, plan, m, q, stack->q_layer_stride, k, v, stack->kv_layer_stride,
                                              kp, vp, stack->prefix_layer_stride, stack->prefix_len, ks, vs,
                                              stack->self_layer_stride, stack->softmax_scale, out, stack->out_layer_stride,
                                              lse, scores, stack->score_accum, workspace, workspace_bytes, stream);
        } else if (stack->k_self) {
            const char* ks = static_cast<const char*>(stack->k_self) + (size_t)c.first * stack->self_layer_stride * esize;
            const char* vs = static_cast<const char*>(stack->v_self) + (size_t)c.first * stack->self_layer_stride * esize;
            rc = cf_query_prefill_attn_full(geom, &local, plan, m, q, stack->q_layer_stride, k, v, stack->kv_layer_stride,
                                            ks, vs, stack->self_layer_stride, stack->softmax_scale, out,
                                            stack->out_layer_stride, lse, scores, stack->score_accum, workspace,
                                            workspace_bytes, stream);
        } else {
            rc = cf_query_prefill_attn_layers(geom, &local, plan, m, q, stack->q_layer_stride, k, v,
                                              stack->kv_layer_stride, stack->softmax_scale, out, stack->out_layer_stride,
                                              lse, scores, stack->score_accum, workspace, workspace_bytes, stream);
        }
        if (rc != CF_OK) return rc;
        if (c.prune_after >= 0) {
            rc = cf_prune_topk(geom, &local, plan, stack->score_accum, stack->prune_keep[c.prune_after], nullptr,
                               stack->strategy, stream);
            if (rc != CF_OK) return rc;
            keep = std::min(keep, stack->prune_keep[c.prune_after]);
            local.tiles_hint = live_tiles_hint(batch, stack, keep);
        }
    }

    // Phase 2: the survivors' keys at their final positions, every layer
    if (stack->k_final) {
        rc = cf_reposition_keys(geom, &local, plan, stack->n_layers, stack->kv_layer_stride, stack->k_cache,
                                stack->k_final, stream);
        if (rc != CF_OK) return rc;
    }
    return CF_OK;
}

int cf_prune_topk_host(int32_t n_docs, const float* score_accum, const int32_t* order, int32_t n_kept, int32_t keep,
                       int32_t strategy, int32_t* order_out, int32_t* n_out) {
    if (n_docs < 0 || n_kept < 0 || n_kept > n_docs || keep < 0 || !n_out || (n_kept > 0 && (!order || !score_accum)))
        return CF_ERR_INVALID_ARG;
    if (strategy != CF_ALLOC_NONE && strategy != CF_ALLOC_ALIGN && strategy != CF_ALLOC_SORT) return CF_ERR_INVALID_ARG;
    std::vector<char> seen((size_t)n_docs, 0);
    for (int r = 0; r < n_kept; ++r) {
        const int i = order[r];
        if (i < 0 || i >= n_docs || seen[i]) return CF_ERR_INVALID_ARG;
        seen[i] = 1;
    }
    const int n_keep = std::min(keep, n_kept);
    if (n_keep > 0 && !order_out) return CF_ERR_INVALID_ARG;
    // rank of a kept document = how many kept documents beat it (larger S; equal S: lower id)
    std::vector<int> by_rank((size_t)n_kept, -1);
    std::vector<char> survives((size_t)n_docs, 0);
    for (int r = 0; r < n_kept; ++r) {
        const int i = order[r];
        int better = 0;
        for (int o = 0; o < n_kept; ++o) {
            const int j = order[o];
            better += (score_accum[j] > score_accum[i]) || (score_accum[j] == score_accum[i] && j < i);
        }
        if (better < n_keep) {
            survives[i] = 1;
            if (better < n_kept) by_rank[better] = i;
        }
    }
    int n = 0;
    if (strategy == CF_ALLOC_SORT) {
        for (int r = 0; r < n_keep; ++r)
            if (by_rank[r] >= 0) order_out[n++] = by_rank[r];
    } else {
        for (int r = 0; r < n_kept; ++r)
            if (survives[order[r]]) order_out[n++] = order[r];
    }
    *n_out = n;
    return CF_OK;
}

int cf_debug_wait_timeout(const cf_geom* geom, const cf_batch* batch, void* plan, int64_t limit_cycles, void* stream) {
    if (!batch || !plan) return CF_ERR_INVALID_ARG;
    int rc = validate(geom, batch);
    if (rc != CF_OK) return rc;
    if (reinterpret_cast<uintptr_t>(plan) % 256 != 0) return CF_ERR_WORKSPACE;
    if (limit_cycles < 1 || limit_cycles > 2000000000LL) return CF_ERR_INVALID_ARG;
    return launch_wait_probe(make_plan_view(geom, batch, plan), limit_cycles, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
