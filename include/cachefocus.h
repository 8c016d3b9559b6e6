/*
 * cachefocus.h -- C ABI of the CacheFocus query-time path for NVIDIA B200 (sm_100a).
 *
 * The library implements the part of CacheFocus (arXiv 2502.11101) that runs between
 * retrieval and decoding: cached per-document keys are moved to new positions by a rotary
 * delta rotation (Sec. 2.3, Eq. 5), the query tokens attend over the concatenated
 * re-positioned document caches (Eq. 1), every document's share of the attention mass is
 * accumulated over layers, and at pruning layers only the best documents survive and are
 * re-allocated next to the query (Sec. 2.4 Algorithm 2, Sec. 2.5).
 *
 * Conventions
 *   - Every function returns CF_OK (0) or a CF_ERR_* code; cf_error_string() names it.
 *   - "host" pointers are ordinary process memory, read or written only during the call.
 *     "device" pointers are CUDA global memory owned by the caller.  The library allocates
 *     and frees no device memory and never synchronises the device, except cf_plan_status()
 *     which copies one word back.
 *   - Device work is queued on `stream` (a cudaStream_t passed as void*, NULL = default
 *     stream) and is asynchronous.  Calls on one stream execute in order.
 *   - Key/value store layout: one layer is `[total_tokens][n_kv_heads][head_dim]` with
 *     `token_stride` elements between rows; the documents of all requests of a batch are
 *     laid end to end; document i owns rows doc_offsets[i] .. doc_offsets[i+1]-1 and its
 *     token t was cached at position doc_src_start[i] + t.  Keys are stored already
 *     rotary-encoded at those positions.  Values are never modified.
 *   - Query/output layout: `[n_requests][q_len][n_q_heads][head_dim]`, contiguous.  The
 *     query states must already be rotary-encoded at positions query_start + j.
 *   - Query head h reads key/value head h / (n_q_heads / n_kv_heads).
 *   - Document ids inside a request are local (0 .. n_b-1); arrays indexed by document use
 *     the global index req_doc_begin[b] + local id.
 */
#ifndef CACHEFOCUS_H_
#define CACHEFOCUS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CF_OK               0
#define CF_ERR_INVALID_ARG  1   /* NULL pointer, negative size, inconsistent geometry            */
#define CF_ERR_RANGE        2   /* the kept documents do not fit the positional range           */
#define CF_ERR_UNSUPPORTED  3   /* head_dim / dtype / layout combination that is not built      */
#define CF_ERR_WORKSPACE    4   /* plan or workspace buffer too small or misaligned             */
#define CF_ERR_CUDA         5   /* a CUDA runtime or driver call failed                         */
#define CF_ERR_TIMEOUT      6   /* a bounded device-side wait expired (reported via the plan)   */

#define CF_BF16 0
#define CF_F32  1

#define CF_ROPE_HALF        0   /* slice p = coordinates (p, p + head_dim/2)                    */
#define CF_ROPE_INTERLEAVED 1   /* slice p = coordinates (2p, 2p + 1)                           */

#define CF_ALLOC_NONE  0        /* survivors keep their positions, gaps stay                    */
#define CF_ALLOC_ALIGN 1        /* Dynamic Positional Allocation ("align", Sec. 2.5)            */
#define CF_ALLOC_SORT  2        /* Attention-Guided Allocation ("sort", Sec. 2.5)               */

#define CF_TILE_TOKENS 128      /* key tiles never straddle two documents                       */
#define CF_MAX_DOCS_PER_REQUEST 1024
#define CF_MAX_SPLITS 64
#define CF_MAX_LAYERS_PER_CALL 64 /* layers one cf_query_prefill_attn_layers call may batch       */
#define CF_STATIC_WORKSPACE_BYTES (32u << 20)   /* scratch carried by cf_query_prefill_attn_static */

/* Model-side geometry.  head_dim 64 or 128; pos_range = the model's positional range L of
 * Eq. 6; rope_theta = base of the rotary frequencies theta^(-2p/head_dim). */
typedef struct cf_geom {
    int32_t n_q_heads;
    int32_t n_kv_heads;
    int32_t head_dim;
    int32_t dtype;        /* CF_BF16 | CF_F32: storage type of Q, K, V and the output */
    int32_t rope_layout;  /* CF_ROPE_HALF | CF_ROPE_INTERLEAVED */
    int32_t pos_range;
    double  rope_theta;
} cf_geom;

/* One batch of independent requests over one packed store.  The three arrays are DEVICE
 * memory and stay owned by the caller; they must remain valid while queued work uses them. */
typedef struct cf_batch {
    int32_t n_requests;
    int32_t n_docs_total;      /* documents of all requests                                      */
    int32_t q_len;             /* query tokens per request                                       */
    int32_t prefix_len;        /* positions [0, prefix_len) are never given to documents         */
    int32_t tail_reserve;      /* positions kept free after query_start (query + new tokens)     */
    int32_t n_reuse;           /* number of parallel windows; 0 = Eq. 6                          */
    int32_t tiles_hint;        /* upper bound of live key tiles per request (0 = derive from
                                  total_tokens); only steers grid sizes, never correctness       */
    int32_t reserved;
    int64_t total_tokens;      /* rows in one layer of the store                                 */
    int64_t token_stride;      /* elements between consecutive rows, >= n_kv_heads*head_dim      */
    const int32_t* req_doc_begin;  /* device [n_requests+1]                                      */
    const int32_t* doc_offsets;    /* device [n_docs_total+1]                                    */
    const int32_t* doc_src_start;  /* device [n_docs_total]                                      */
} cf_batch;

/* Byte offsets of the fields inside a plan buffer (device memory written by cf_plan_init and
 * cf_prune_topk, read by the other device calls).  All int32 unless noted. */
typedef struct cf_plan_layout {
    size_t total_bytes;
    size_t status;          /* [4]   status[0] = first CF_ERR_* raised on the device, 0 if none  */
    size_t kept;            /* [n_docs_total] local ids by rank, request b starts at
                                     req_doc_begin[b]; rank 0 sits next to the query              */
    size_t kept_count;      /* [n_requests]                                                      */
    size_t dst_start;       /* [n_docs_total] destination position of token 0, -1 if pruned      */
    size_t group;           /* [n_docs_total] window index, -1 if pruned                         */
    size_t n_reuse;         /* [n_requests]                                                      */
    size_t query_start;     /* [n_requests]                                                      */
    size_t n_tiles;         /* [n_requests]                                                      */
    size_t tile_begin;      /* [n_requests] first tile slot of the request (index into tile_*)   */
    size_t doc_tile_begin;  /* [n_docs_total] first tile of the document (index into tile_*)     */
    size_t doc_tile_count;  /* [n_docs_total] 0 if pruned                                        */
    size_t tile_doc;        /* [max_tiles] global document index                                 */
    size_t tile_row0;       /* [max_tiles] first store row                                       */
    size_t tile_len;        /* [max_tiles] 1..CF_TILE_TOKENS                                     */
    size_t trig;            /* float [n_docs_total][head_dim/2][2] = cos, sin of delta*freq      */
    int32_t max_tiles;
    int32_t reserved;
} cf_plan_layout;

const char* cf_error_string(int code);

/* ---------------------------------------------------------------- host-side integer steps */

/* Adaptive Re-Positioning (Sec. 2.3.1, Eq. 6) and Adaptive Positional Allocation (Sec. 2.5)
 * for ONE request, on the host.  All pointers are host memory.
 *   doc_len[n_docs]   token count of every document of the request
 *   order[n_kept]     distinct document ids; order[0] is placed closest to the query
 *   n_reuse           >0 forces the number of parallel windows, 0 selects
 *                     ceil(n_kept / floor(capacity / l_C)) with l_C = longest kept document and
 *                     capacity = pos_range - prefix_len - tail_reserve
 *   query_start       <0: the query closes the usable range (pos_range - tail_reserve)
 * Rank r goes to window r mod n_reuse; inside a window documents take sequential positions,
 * packed backwards from query_start.  Outputs: dst_start[n_docs], group[n_docs] (-1 for
 * documents not in `order`), *n_reuse_out, *query_start_out (either may be NULL).
 * Errors: CF_ERR_INVALID_ARG (bad ids, empty documents), CF_ERR_RANGE (does not fit). */
int cf_allocate_positions(const cf_geom* geom, int32_t n_docs, const int32_t* doc_len,
                          const int32_t* order, int32_t n_kept, int32_t prefix_len,
                          int32_t tail_reserve, int32_t n_reuse, int32_t query_start,
                          int32_t* dst_start, int32_t* group, int32_t* n_reuse_out,
                          int32_t* query_start_out);

/* Linear pruning schedule of App. C: pruning after every `every`-th layer (1-based),
 * k_prune = (k - k_finish) / (n_layers / every) documents each time, any remainder removed at
 * the last pruning layer.  Writes up to `capacity` (layer, keep) pairs into host arrays and the
 * number of pruning layers into *count. */
int cf_schedule_linear(int32_t n_layers, int32_t every, int32_t k, int32_t k_finish,
                       int32_t capacity, int32_t* layers, int32_t* keeps, int32_t* count);

/* ------------------------------------------------------------------------ device-side plan */

/* Field offsets and size of the plan buffer for this geometry and batch (host computation). */
int cf_plan_layout_of(const cf_geom* geom, const cf_batch* batch, cf_plan_layout* layout);

/* Start a request batch (Algorithm 2, "Init"): sets the kept list of every request from
 * `order` (device [n_docs_total], local ids by rank laid out like `kept`; NULL = identity,
 * i.e. retrieval order) and `kept_count` (device [n_requests]; NULL = all documents), then
 * allocates positions (same rules as cf_allocate_positions, query_start < 0 = end of range),
 * and derives per-document rotation tables and the key-tile list.  `plan` is device memory of
 * at least cf_plan_layout.total_bytes bytes, 256-byte aligned.  Device-side failures (range
 * overflow) are recorded in the plan's status word. */
int cf_plan_init(const cf_geom* geom, const cf_batch* batch, const int32_t* order,
                 const int32_t* kept_count, int32_t query_start, void* plan, size_t plan_bytes,
                 void* stream);

/* Copies the plan's status word back (synchronises `stream`); returns it as the error code. */
int cf_plan_status(const cf_geom* geom, const cf_batch* batch, const void* plan, void* stream);

/* ------------------------------------------------------------------------------ hot path */

/* Cache Re-Positioning (Eq. 5; Algorithm 2 Phase 2): for every kept document of the plan and
 * every layer, rotates each two-dimensional slice of each key row by the angle of
 * (dst_start - src_start) positions and writes it to k_out (same layout; k_out may equal k_in;
 * rows of pruned documents are not written).  `n_layers` layers are processed,
 * `layer_stride` elements apart.  Arithmetic: fp32, one rounding to the storage type. */
int cf_reposition_keys(const cf_geom* geom, const cf_batch* batch, const void* plan,
                       int32_t n_layers, int64_t layer_stride, const void* k_in, void* k_out,
                       void* stream);

/* Attention over the union of two disjoint key sets from the attention over each (Eq. 1 is a softmax,
 * so two results combine through their log-sum-exp): for instance the kept documents and a pinned
 * segment such as the shared prefix cache C_prefix of Algorithm 2, which is attended by a call of its
 * own (a batch whose only "document" is the prefix, cached and kept at the same positions, so its
 * delta is 0; it is in no kept list, hence never pruned, and the documents' scores are untouched).
 *   out_a, out_b, out  device [n_blocks][q_len][n_q_heads][head_dim], storage type (out may be out_a or out_b)
 *   lse_a, lse_b, lse  device float [n_blocks][n_q_heads][q_len], natural log; lse may be NULL, lse_a or lse_b
 *   n_blocks           layers x requests covered by the buffers */
int cf_merge_attn(const cf_geom* geom, int32_t n_blocks, int32_t q_len, const void* out_a, const float* lse_a,
                  const void* out_b, const float* lse_b, void* out, float* lse, void* stream);

/* Algorithm 2, Phase 2, assembled (C_final): for every layer and request, the re-positioned keys
 * (Eq. 5) and the values of the surviving documents, packed in rank order (rank 0 first), followed by
 * the query tokens' own keys and values (C_Q^l, unchanged).
 *   k_cache, v_cache  the store, n_layers layers, layer_stride elements apart (as cf_reposition_keys)
 *   k_self, v_self    [n_layers][n_requests][q_len][n_kv_heads][head_dim], self_layer_stride apart
 *   k_out, v_out      device [n_layers][n_requests][out_rows][n_kv_heads][head_dim], dense; request b
 *                     receives final_rows[b] rows per layer, rows beyond stay untouched
 *   final_rows        device int32 [n_requests]: tokens of the survivors + q_len
 * A request whose rows do not fit out_rows raises CF_ERR_WORKSPACE in the plan's status word; its
 * final_rows entry is not written, the leading tiles that do fit may have been copied, and nothing
 * is ever written beyond out_rows. */
int cf_assemble_final_cache(const cf_geom* geom, const cf_batch* batch, const void* plan,
                            int32_t n_layers, int64_t layer_stride, const void* k_cache, const void* v_cache,
                            int64_t self_layer_stride, const void* k_self, const void* v_self,
                            int32_t out_rows, void* k_out, void* v_out, int32_t* final_rows, void* stream);

/* Scratch needed by cf_query_prefill_attn for this batch (bytes; 256-byte aligned buffer).
 * Grows with batch->tiles_hint: ask with the largest hint that will be used. */
size_t cf_attn_workspace_bytes(const cf_geom* geom, const cf_batch* batch);

/* One layer of query-token attention over the kept documents' caches (Eq. 1; Algorithm 2,
 * "layer_l" restricted to its attention over the cached documents), fused with the
 * re-positioning of the keys (Eq. 5): keys are read from the un-repositioned store `k_cache`
 * and rotated on the way in.
 *   q, out        device [n_requests][q_len][n_q_heads][head_dim], storage type
 *   k_cache, v_cache  device, one layer of the store
 *   softmax_scale 0 selects 1/sqrt(head_dim)
 *   lse           device float [n_requests][n_q_heads][q_len], natural log of the softmax
 *                 denominator (lets the caller merge further key blocks); may be NULL
 *   doc_scores    device float [n_docs_total]: share of the attention mass on each document,
 *                 averaged over heads and query rows (sums to 1 per request, 0 for pruned
 *                 documents); may be NULL
 *   score_accum   device float [n_docs_total], += doc_scores (Algorithm 2: S <- S + s^l);
 *                 may be NULL
 * Accumulation is fp32; reductions run in a fixed order (results are run-to-run identical). */
int cf_query_prefill_attn(const cf_geom* geom, const cf_batch* batch, const void* plan,
                          const void* q, const void* k_cache, const void* v_cache,
                          float softmax_scale, void* out, float* lse, float* doc_scores,
                          float* score_accum, void* workspace, size_t workspace_bytes,
                          void* stream);

/* Several consecutive layers that attend the same kept documents, in one call (Algorithm 2:
 * between two pruning layers the set ids, and with it the allocation, does not change, so
 * layer_l ... layer_{l+m-1} read one plan).  Equivalent to n_layers successive calls of
 * cf_query_prefill_attn on layer slices of the arguments, S <- S + s^l accumulated in layer
 * order; the layers run side by side on the device.  A caller can use it when the query states
 * of those layers are available together (replay, benchmarking, scoring passes with stored
 * queries); inside a running model each layer's queries depend on the previous layer's output,
 * and the single-layer call is the one that applies.
 *   n_layers          1 .. CF_MAX_LAYERS_PER_CALL, and n_layers * n_requests <= 65535
 *   q, out            layer i at q + i * q_layer_stride, out + i * out_layer_stride (elements);
 *                     each layer laid out as in cf_query_prefill_attn
 *   k_cache, v_cache  layer i of the store at + i * kv_layer_stride elements (a multiple of 8
 *                     bf16 / 4 fp32 elements, at least total_tokens * token_stride if n_layers > 1)
 *   lse               float [n_layers][n_requests][n_q_heads][q_len] or NULL
 *   doc_scores        float [n_layers][n_docs_total] or NULL (every layer's s^l)
 *   score_accum       float [n_docs_total] or NULL
 *   workspace         at least cf_attn_workspace_bytes_layers(geom, batch, n_layers) bytes */
size_t cf_attn_workspace_bytes_layers(const cf_geom* geom, const cf_batch* batch, int32_t n_layers);
int cf_query_prefill_attn_layers(const cf_geom* geom, const cf_batch* batch, const void* plan,
                                 int32_t n_layers, const void* q, int64_t q_layer_stride,
                                 const void* k_cache, const void* v_cache, int64_t kv_layer_stride,
                                 float softmax_scale, void* out, int64_t out_layer_stride,
                                 float* lse, float* doc_scores, float* score_accum,
                                 void* workspace, size_t workspace_bytes, void* stream);

/* One layer at a time with the document scores deferred (Algorithm 2 uses S only where it prunes: S <- S + s^l of
 * the layers since the last cut can be added together right before the next one).  For a running model, whose
 * layers come one by one: cf_query_prefill_attn_slot is cf_query_prefill_attn for one layer without doc_scores and
 * score_accum -- it leaves the layer's per-tile and per-row log-sum-exps in slot `slot` of the workspace --, and
 * cf_accumulate_scores then does for slots 0 .. n_filled-1 what the attention calls would have done: doc_scores[i] =
 * s of slot i (optional), S <- S + s in slot order (the per-layer calls' values up to the rounding of fp32 sums
 * taken in another order; run-to-run identical).  Between the first slot
 * call and cf_accumulate_scores the plan must not change (no cf_prune_topk), and every slot 0 .. n_filled-1 must
 * have been filled; the slot calls of one workspace must not overlap on the device (they share its partial-result
 * buffers).  One launch chain of two kernels per layer instead of three.
 *   slot, n_slots   0 <= slot < n_slots <= CF_MAX_LAYERS_PER_CALL, n_slots * n_requests <= 65535; n_slots is the
 *                   capacity the workspace is laid out for, the same in every call of the group
 *   n_filled        1 .. n_slots: slots to score
 *   workspace       at least cf_attn_workspace_bytes_slots(geom, batch, n_slots) bytes, the same buffer in every call
 *   doc_scores      device float [n_filled][n_docs_total] or NULL;  score_accum  device float [n_docs_total] or NULL
 * Errors as cf_query_prefill_attn. */
size_t cf_attn_workspace_bytes_slots(const cf_geom* geom, const cf_batch* batch, int32_t n_slots);
int cf_query_prefill_attn_slot(const cf_geom* geom, const cf_batch* batch, const void* plan, int32_t slot,
                               int32_t n_slots, const void* q, const void* k_cache, const void* v_cache,
                               float softmax_scale, void* out, float* lse, void* workspace, size_t workspace_bytes,
                               void* stream);
int cf_accumulate_scores(const cf_geom* geom, const cf_batch* batch, const void* plan, int32_t n_filled, int32_t n_slots,
                         float* doc_scores, float* score_accum, void* workspace, size_t workspace_bytes, void* stream);
/* The slot call with the key blocks besides the documents (one layer of cf_query_prefill_attn_prefix without the
 * scores): a shared prefix cache (prefix_len > 0; k_prefix, v_prefix [prefix_len][n_kv_heads][head_dim]) and / or the
 * query tokens' own keys and values (k_self, v_self [n_requests][q_len][n_kv_heads][head_dim]; both NULL: none); at
 * least one of the two.  Its workspace is larger (cf_attn_workspace_bytes_slots_full); cf_accumulate_scores reads
 * either kind. */
size_t cf_attn_workspace_bytes_slots_full(const cf_geom* geom, const cf_batch* batch, int32_t n_slots);
int cf_query_prefill_attn_slot_full(const cf_geom* geom, const cf_batch* batch, const void* plan, int32_t slot,
                                    int32_t n_slots, const void* q, const void* k_cache, const void* v_cache,
                                    const void* k_prefix, const void* v_prefix, int32_t prefix_len, const void* k_self,
                                    const void* v_self, float softmax_scale, void* out, float* lse, void* workspace,
                                    size_t workspace_bytes, void* stream);

/* The whole attention of the query tokens in layer_l (Algorithm 2): over the kept documents' caches
 * as in cf_query_prefill_attn_layers, and over the query tokens themselves under the causal mask
 * that the footnote to Eq. 1 refers to (query row j sees query tokens 0..j), merged into one softmax.
 *   k_self, v_self  device, keys and values of the query tokens, keys already encoded at
 *                   query_start + j: layer i at + i * self_layer_stride elements, each layer
 *                   [n_requests][q_len][n_kv_heads][head_dim]; q_len <= 128
 *   out, lse        cover both key sets (lse = log of the joint denominator)
 *   doc_scores, score_accum  as in cf_query_prefill_attn: the documents' shares of the mass that falls
 *                   on the documents (they still sum to 1 per request), so pruning decisions do not
 *                   depend on whether the caller merges the query-self block here or elsewhere
 *   workspace       at least cf_attn_workspace_bytes_full(geom, batch, n_layers) bytes */
size_t cf_attn_workspace_bytes_full(const cf_geom* geom, const cf_batch* batch, int32_t n_layers);
int cf_query_prefill_attn_full(const cf_geom* geom, const cf_batch* batch, const void* plan,
                               int32_t n_layers, const void* q, int64_t q_layer_stride,
                               const void* k_cache, const void* v_cache, int64_t kv_layer_stride,
                               const void* k_self, const void* v_self, int64_t self_layer_stride,
                               float softmax_scale, void* out, int64_t out_layer_stride,
                               float* lse, float* doc_scores, float* score_accum,
                               void* workspace, size_t workspace_bytes, void* stream);

/* cf_query_prefill_attn_full with the shared prefix cache C_prefix attended in the same call
 * (Algorithm 2: concat([C_prefix] + [C_d_i ...]); Sec. 2.2: every document was cached behind that prefix):
 * the prefix's keys are used as cached, at positions 0 .. prefix_len-1 (delta 0, no rotation), every query row
 * sees all of them, and they ride along as further key tiles of the same kernel.  The prefix is no document: it
 * is in no kept list, never pruned, and doc_scores stay the documents' shares of the mass that falls on the
 * documents (they still sum to 1 per request); out and lse cover all key sets.
 *   k_prefix, v_prefix  device [n_layers][prefix_len][n_kv_heads][head_dim] dense, layers prefix_layer_stride
 *                   elements apart; one prefix for all requests of the batch; prefix_len <= batch->prefix_len
 *                   (the positions the allocation keeps clear of documents)
 *   k_self, v_self  as in cf_query_prefill_attn_full, or both NULL: documents and prefix only
 *   workspace       at least cf_attn_workspace_bytes_full(geom, batch, n_layers) bytes
 * With bf16 storage and head_dim 128 the prefix rides along as key tiles of the tensor-core kernel; other geometries
 * compute it (and the query-self block) as one more part of the split-KV merge on the CUDA cores. */
int cf_query_prefill_attn_prefix(const cf_geom* geom, const cf_batch* batch, const void* plan,
                                 int32_t n_layers, const void* q, int64_t q_layer_stride,
                                 const void* k_cache, const void* v_cache, int64_t kv_layer_stride,
                                 const void* k_prefix, const void* v_prefix, int64_t prefix_layer_stride,
                                 int32_t prefix_len, const void* k_self, const void* v_self,
                                 int64_t self_layer_stride, float softmax_scale, void* out,
                                 int64_t out_layer_stride, float* lse, float* doc_scores, float* score_accum,
                                 void* workspace, size_t workspace_bytes, void* stream);

/* The same computation as cf_query_prefill_attn for callers that cannot allocate device memory
 * (the paper has no counterpart; this is a property of the library, not of the method).
 * Who needs it: code that runs where cudaMalloc is off limits -- a plugin inside a host
 * application that owns the allocator and hands out only input and output buffers, a serving
 * loop that has frozen its memory pool, a caller already inside a region where allocation would
 * synchronise the device.  Such a caller has nowhere to put the attention workspace, so here the
 * workspace is a fixed array of CF_STATIC_WORKSPACE_BYTES (32 MiB) that is part of the library
 * image: every GPU that loads the library holds those bytes until the process exits.
 *   - Arguments are those of cf_query_prefill_attn without workspace / workspace_bytes.
 *   - Returns CF_ERR_WORKSPACE, launching nothing, when cf_attn_workspace_bytes(geom, batch) for
 *     this batch exceeds CF_STATIC_WORKSPACE_BYTES.  Use a smaller batch or the ordinary call.
 *   - The first call on each device looks up the array's device address (one
 *     cudaGetSymbolAddress); make that first call outside any stream capture.  No call allocates
 *     or frees device memory.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left.
 *     Nothing in it has to start at zero: each call overwrites every word it later reads.  Two
 *     calls that run on the GPU at the same time (different streams, or different host threads)
 *     would overwrite each other's partial results: issue them on one stream, or otherwise make
 *     sure they do not overlap. */
int cf_query_prefill_attn_static(const cf_geom* geom, const cf_batch* batch, const void* plan,
                                 const void* q, const void* k_cache, const void* v_cache,
                                 float softmax_scale, void* out, float* lse, float* doc_scores,
                                 float* score_accum, void* stream);

/* Layer-Adaptive Cache Pruning step (Algorithm 2: argsort of S, prun) followed by the
 * re-allocation of the survivors (Sec. 2.5), all on the device: per request keeps the `keep`
 * documents with the largest score_accum among the kept ones (ties: lower id), orders them
 * (ALIGN/NONE: previous order, SORT: by score, best first), re-allocates positions with the
 * request's query_start unchanged (NONE: positions untouched) and rebuilds rotation tables and
 * tile list in `plan`.  keep_per_request (device [n_requests]) overrides `keep` when not NULL. */
int cf_prune_topk(const cf_geom* geom, const cf_batch* batch, void* plan,
                  const float* score_accum, int32_t keep, const int32_t* keep_per_request,
                  int32_t strategy, void* stream);

/* ------------------------------------------------------------------------------- decoding
 * Algorithm 2, Phase 3 (Y <- LLM(C_final)) and the "Decoding" loop of Algorithm 1: every generated
 * token appends its key/value rows to each request's final cache and attends all of its rows; the cost
 * is the O((2 l_c n + a) a / 2) term of Sec. 3.3 and the decode columns of Table 2.  The caches are the
 * packed buffers cf_assemble_final_cache writes, [n_layers][n_requests][cache_rows][n_kv_heads][head_dim]
 * with request b using its first rows[b] rows (`rows` = that call's final_rows, device int32
 * [n_requests], never modified here).  Their keys are already re-positioned, so nothing is rotated; the
 * new token's key must come rotary-encoded at its own position.  A step t = 0, 1, ... of the loop is
 *     cf_decode_append(..., rows, t, k_new, v_new, ...)      rows[b] + t receives the new rows
 *     cf_decode_plan(..., rows, t + 1, decode_plan, ...)     once per step: rows[b] + t + 1 rows in use
 *     cf_decode_attn(..., decode_plan, ...)                  per layer, or for several layers at once
 * All three are asynchronous on `stream`.  cache_rows is the row capacity of a request's slot. */

/* Bytes of the decode-plan buffer (device memory, 256-byte aligned) for this batch shape. */
size_t cf_decode_plan_bytes(const cf_geom* geom, int32_t n_requests, int32_t cache_rows);

/* Describes one decoding step to the attention kernels: request b attends rows 0 .. rows[b] +
 * extra_rows - 1 of its slot.  A request whose count is below 1 or above cache_rows raises CF_ERR_RANGE
 * in the buffer's status word (read it with cf_decode_status) and is clamped. */
int cf_decode_plan(const cf_geom* geom, int32_t n_requests, int32_t cache_rows, const int32_t* rows,
                   int32_t extra_rows, void* decode_plan, size_t decode_plan_bytes, void* stream);

/* Copies the status word of a decode plan back (synchronises `stream`); returns it as the error code. */
int cf_decode_status(const cf_geom* geom, int32_t n_requests, int32_t cache_rows, const void* decode_plan,
                     void* stream);

/* Scratch of cf_decode_attn for calls over up to n_layers layers. */
size_t cf_decode_workspace_bytes(const cf_geom* geom, int32_t n_requests, int32_t cache_rows, int32_t n_layers);

/* The new token's attention (Eq. 1, one query row per head) over the rows the decode plan names.
 *   q, out    device [n_layers][n_requests][n_q_heads][head_dim], layers q_layer_stride / out_layer_stride
 *             elements apart (n_layers = 1 inside a running model: layer l+1's query comes out of layer l)
 *   k_final, v_final  the final caches, layers kv_layer_stride elements apart
 *   lse       device float [n_layers][n_requests][n_q_heads] or NULL
 *   workspace at least cf_decode_workspace_bytes(..., n_layers) bytes, 256-byte aligned */
int cf_decode_attn(const cf_geom* geom, int32_t n_requests, int32_t cache_rows, const void* decode_plan,
                   int32_t n_layers, const void* q, int64_t q_layer_stride, const void* k_final,
                   const void* v_final, int64_t kv_layer_stride, float softmax_scale, void* out,
                   int64_t out_layer_stride, float* lse, void* workspace, size_t workspace_bytes, void* stream);

/* Appends one token per request: row rows[b] + step of request b's slot receives k_new / v_new
 * ([n_layers][n_requests][n_kv_heads][head_dim], layers new_layer_stride elements apart) in every layer.
 * A request without room raises CF_ERR_RANGE in *status (device int32, may be NULL; only written on
 * failure) and is skipped. */
int cf_decode_append(const cf_geom* geom, int32_t n_requests, int32_t cache_rows, int32_t n_layers,
                     void* k_final, void* v_final, int64_t kv_layer_stride, const int32_t* rows, int32_t step,
                     const void* k_new, const void* v_new, int64_t new_layer_stride, int32_t* status, void* stream);

/* A batch of documents for the offline cache construction: a packed store like cf_batch's, without
 * requests, allocation or plan.  doc_offsets is DEVICE memory owned by the caller. */
typedef struct cf_doc_batch {
    int32_t n_docs;
    int32_t max_doc_len;      /* upper bound of the documents' token counts (sizes the grid; a document
                                 longer than this is only partly processed)                           */
    int32_t prefix_len;       /* tokens of the shared prefix cache, 0 = none                          */
    int32_t reserved;
    int64_t total_tokens;     /* rows of one layer of the packed tensors                              */
    int64_t token_stride;     /* elements between consecutive key/value rows, >= n_kv_heads*head_dim  */
    const int32_t* doc_offsets;   /* device [n_docs+1]: document i owns rows doc_offsets[i] .. [i+1]-1 */
} cf_doc_batch;

/* Attention of the offline, query-independent cache construction C_d <- LLM(C_prefix, d) (Sec. 2.2;
 * the O(l_c^2 k) term of the complexity paragraph in Sec. 3.3): in every layer, token t of a document
 * attends the shared prefix cache and the document's own tokens 0..t (causal mask of Eq. 1); documents
 * are processed in parallel and do not see each other.  Queries and keys are used as given: the
 * caller has already rotary-encoded them (prefix at positions 0..prefix_len-1, every document right
 * behind it), so no re-positioning happens here; the keys and values passed in ARE the document
 * caches that the query-time calls above later consume.
 *   q, out          device [n_layers][total_tokens][n_q_heads][head_dim], layers q_layer_stride /
 *                   out_layer_stride elements apart
 *   k, v            device [n_layers][total_tokens][n_kv_heads][head_dim] with docs->token_stride
 *                   between rows, layers kv_layer_stride elements apart
 *   k_prefix, v_prefix  device [n_layers][prefix_len][n_kv_heads][head_dim] dense, layers
 *                   prefix_layer_stride elements apart; ignored when prefix_len = 0
 *   softmax_scale   0 selects 1/sqrt(head_dim)
 *   lse             device float [n_layers][n_q_heads][total_tokens], natural log of each row's softmax
 *                   denominator; may be NULL
 *   status          device int32 or NULL: receives CF_ERR_TIMEOUT if a bounded device-side wait of the
 *                   tensor-core kernel expired (it is only ever written on failure: clear it first)
 * Needs no workspace.  Errors: CF_ERR_INVALID_ARG (null or misaligned pointers, strides). */
int cf_document_prefill_attn(const cf_geom* geom, const cf_doc_batch* docs, int32_t n_layers,
                             const void* q, int64_t q_layer_stride, const void* k, const void* v,
                             int64_t kv_layer_stride, const void* k_prefix, const void* v_prefix,
                             int64_t prefix_layer_stride, float softmax_scale, void* out,
                             int64_t out_layer_stride, float* lse, int32_t* status, void* stream);

/* Host-side mirror of the pruning step alone (Algorithm 2: argsort of S, prun), integers and scores
 * in host memory, nothing launched: among the documents of `order` (n_kept distinct local ids, rank
 * order) keeps the min(keep, n_kept) with the largest score_accum[id] (ties: lower id) and writes
 * them to order_out (capacity min(keep, n_kept)): in their previous relative order for CF_ALLOC_NONE
 * and CF_ALLOC_ALIGN, best first for CF_ALLOC_SORT.  *n_out receives their number.  The device call
 * cf_prune_topk takes the same decisions; this one serves callers that hold S on the host, and tests. */
int cf_prune_topk_host(int32_t n_docs, const float* score_accum, const int32_t* order, int32_t n_kept,
                       int32_t keep, int32_t strategy, int32_t* order_out, int32_t* n_out);

/* Algorithm 2, Phases 1 and 2, for a whole layer stack whose per-layer query states are given up
 * front (benchmarks, replay, scoring passes with stored queries; inside a running model layer l+1's
 * queries come out of layer l, and the per-layer calls above apply).  The struct is host memory read
 * during the call; the buffers it names are device memory unless marked host. */
typedef struct cf_stack {
    int32_t n_layers;
    int32_t n_prune;              /* pruning layers in the schedule                                   */
    const int32_t* prune_layer;   /* host [n_prune]: 1-based layers, strictly ascending; pruning
                                     happens after that layer's scores are accumulated                */
    const int32_t* prune_keep;    /* host [n_prune]: documents kept per request from then on          */
    int32_t strategy;             /* CF_ALLOC_NONE | CF_ALLOC_ALIGN | CF_ALLOC_SORT                   */
    int32_t batch_layers;         /* 0: one attention launch chain per layer (the layers' scores wait in
                                     workspace slots and are added to S before each pruning layer:
                                     cf_query_prefill_attn_slot[_full], cf_accumulate_scores);
                                     1: one chain per run of layers between two pruning layers (same
                                     results up to the tolerance of the split-KV merge)               */
    float   softmax_scale;        /* 0 selects 1/sqrt(head_dim)                                       */
    int32_t reserved;
    const void* q;                /* [n_layers][n_requests][q_len][n_q_heads][head_dim]               */
    int64_t q_layer_stride;       /* elements between layers, as in cf_query_prefill_attn_layers      */
    const void* k_cache;          /* the store, n_layers layers                                       */
    const void* v_cache;
    int64_t kv_layer_stride;
    const void* k_self;           /* NULL, or the query tokens' own keys/values: every layer then     */
    const void* v_self;           /* also attends the causal query-self block (..._attn_full)         */
    int64_t self_layer_stride;
    void*   out;                  /* [n_layers][n_requests][q_len][n_q_heads][head_dim]               */
    int64_t out_layer_stride;
    float*  lse;                  /* [n_layers][n_requests][n_q_heads][q_len] or NULL                 */
    float*  layer_scores;         /* [n_layers][n_docs_total] every layer's s^l, or NULL              */
    float*  score_accum;          /* [n_docs_total] S: cleared by the call, holds the sums at the end */
    void*   k_final;              /* NULL, or a store-shaped buffer that receives Phase 2 (may be
                                     k_cache itself)                                                  */
    const int32_t* doc_len_host;        /* host [n_docs_total] or NULL: lets the call size its grids  */
    const int32_t* req_doc_begin_host;  /* host [n_requests+1] or NULL    to the documents still kept */
    const void* k_prefix;         /* NULL, or the shared prefix cache attended by every layer         */
    const void* v_prefix;         /* (cf_query_prefill_attn_prefix): [n_layers][prefix_len][kv][dim]  */
    int64_t prefix_layer_stride;
    int32_t prefix_len;           /* 0 = no prefix; at most batch->prefix_len                         */
    int32_t reserved2;
} cf_stack;

/* Scratch needed by cf_run_stack (the largest of its attention calls); 0 on invalid arguments. */
size_t cf_run_stack_workspace_bytes(const cf_geom* geom, const cf_batch* batch, const cf_stack* stack);

/* Runs Init (S = 0, every document kept in retrieval order, first allocation), then for l = 1..L
 * layer_l's attention over the kept caches with S <- S + s^l and, after a scheduled layer, argsort /
 * prun / re-allocation; finally Phase 2 if k_final is given.  Everything is queued on `stream`; the
 * plan holds the final kept lists and positions afterwards.  Equivalent to the sequence
 * cf_plan_init, cf_query_prefill_attn[_layers|_full] ..., cf_prune_topk ..., cf_reposition_keys. */
int cf_run_stack(const cf_geom* geom, const cf_batch* batch, const cf_stack* stack, void* plan,
                 size_t plan_bytes, void* workspace, size_t workspace_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* CACHEFOCUS_H_ */
