// Fused re-position + query-prefill attention on the Blackwell tensor cores (bf16, head_dim 128).
//
// Eq. 5 fused into Eq. 1: key tiles are streamed from the un-repositioned store by TMA into
// 128B-swizzled shared memory, every key is rotated by its document's delta in registers and
// written back in place, QK^T and PV run as tcgen05.mma with fp32 accumulators in tensor memory,
// the softmax runs one query row per thread out of tensor memory and hands P back through tensor
// memory (bf16, aliased onto the upper half of S).  The cache is read once.
//
// One CTA owns a (layer, request, kv head, group of <=256 query rows, range of key tiles).  Two softmax
// warpgroups work side by side, each with its own S and O accumulators in tensor memory:
//   - with more than 128 query rows in the group, warpgroup w owns row tile w and both see every
//     key tile of the CTA's range;
//   - with at most 128 rows, both own the same rows and take alternate key tiles, i.e. the CTA
//     produces two independent parts of the split-KV decomposition.
// Partial results (reference maximum, sum, unnormalised O) go to the workspace and are merged by
// the combine kernel.  Warp roles (512 threads):
//   warps 0-3    softmax warpgroup 0 (thread = query row = TMEM lane)
//   warps 4-7    softmax warpgroup 1
//   warps 8-11, 14, 15  key rotation in shared memory
//   warp 12      TMA producer (one lane)     warp 13  TMEM allocation and MMA issue (one lane)
// The MMA warp interleaves the two warpgroups (PV of one, then the next QK^T of the same one), so
// one warpgroup's exponentials overlap the other's tensor-core work.
// The softmax is single-pass: the reference maximum of a row only moves when a 32-key chunk exceeds
// it by more than 2^8, in which case O, the sums and the P columns already written are rescaled
// (rare after the first chunk); any reference within the exponent range is exact enough because
// P (bf16) and the sums (fp32) keep their relative precision.
// Every wait on an mbarrier is bounded; when a wait expires the CTA raises CF_ERR_TIMEOUT in the
// plan's status word, all roles leave their loops, and the CTA frees its tensor memory and exits.
#include <algorithm>

#include "cf_tc_util.cuh"

namespace cf {

namespace {

using namespace tc;

constexpr int kThreads = 512;

// Tensor maps of the key store and of the value store, one per box height: a tile is fetched by
// two bulk copies (one per 64-column half) whatever its length.
struct StoreMaps {
    CUtensorMap k[4], v[4];
    CUtensorMap ks[4], vs[4];      // keys and values of the query tokens themselves (calls with a query-self block)
    CUtensorMap kp[4], vp[4];      // keys and values of a shared prefix cache (calls that attend one)
};
constexpr int kSmemTiles = 7;                      // 2 Q + 5 ring, or 1 Q + 6 ring
constexpr int kMetaTiles = 128;                    // key tiles of a CTA whose description is staged in shared memory
constexpr int kSmemBytes = kSmemTiles * kTileBytes + 1024 + 512 + kMetaTiles * 8;   // tiles, alignment slack, barriers, tile list
constexpr int kMaxStages = 6;
constexpr int kRotateThreads = 192;
constexpr float kRescaleThreshold = 8.0f;          // log2 units: the reference maximum moves only
                                                   // when a tile exceeds it by more than 2^8

struct Barriers {
    // A parity wait is only meaningful for a waiter that has seen every earlier phase of the barrier.
    // Key loads and value loads of a ring stage therefore complete on separate barriers: the rotation
    // warps wait for every key load, the MMA warp for every value load.
    unsigned long long kv_full[kMaxStages][2];   // [stage][0 = keys, 1 = values]
    unsigned long long kv_empty[kMaxStages];
    unsigned long long k_ready[kMaxStages];
    unsigned long long s_full[2];
    unsigned long long p_ready[2];
    unsigned long long o_done[2];
    unsigned int tmem_base;
    volatile int abort_flag;
};

static_assert(sizeof(Barriers) <= 512, "barrier block must fit its reserved shared memory");
static_assert(kSmemBytes <= 227 * 1024, "shared memory of one CTA");

// A key tile of the CTA's range: first store row, length, document.  The first kMetaTiles come
// from shared memory (copied there once), later ones from the plan.
struct TileInfo {
    int row0, len, doc;
};
// Key blocks besides the kept documents, which the CTA of the last pair of parts takes after its documents'
// tiles: first the tiles of a shared prefix cache (document -2: rows of the prefix tensors, every row of
// the query sees them), then the query-self block as one tile (document -1: rows of the query's own
// key/value tensors under the causal mask).  Neither is rotated, neither is a document that is scored.
struct ExtraTiles {
    int first;               // index of the first such tile in the CTA's list = number of its document tiles
    int n_prefix, prefix_len;
    int self_it, self_row0, self_len;
};
__device__ __forceinline__ TileInfo tile_info(const int2* s_meta, const PlanView& pv, int ti0, int it, const ExtraTiles& ex) {
    TileInfo t;
    if (it >= ex.first) {
        if (it == ex.self_it) {
            t.row0 = ex.self_row0;
            t.len = ex.self_len;
            t.doc = -1;
        } else {
            t.row0 = (it - ex.first) * kTile;
            t.len = min(kTile, ex.prefix_len - t.row0);
            t.doc = -2;
        }
    } else if (it < kMetaTiles) {
        const int2 m = s_meta[it];
        t.row0 = m.x;
        t.len = m.y & 0xff;
        t.doc = m.y >> 8;
    } else {
        t.row0 = pv.tile_row0[ti0 + it];
        t.len = pv.tile_len[ti0 + it];
        t.doc = pv.tile_doc[ti0 + it];
    }
    return t;
}

// The ring has six stages (one query tile in shared memory) or five (two query tiles); dividing by
// a literal keeps the index arithmetic of the hot loops to a few instructions.
__device__ __forceinline__ int ring_mod(int x, bool six) { return six ? x % 6 : x % 5; }
__device__ __forceinline__ int ring_div(int x, bool six) { return six ? x / 6 : x / 5; }
// Loads of one kind (keys or values) a stage has received before the one of tile `it`.
__device__ __forceinline__ int ring_uses(int it, bool six) { return six ? it / 3 : it / 5; }

// ROTATE = false: every document sits where it was cached (the final caches of a decoding step), so the keys go from
// the copy straight to the tensor cores and the rotation warps stay idle.
template <int LAYOUT, bool ROTATE>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ StoreMaps maps,
               BatchView bv, PlanView pv, AttnWorkspace ws, long long q_layer_stride, int n_q_heads, int n_kv_heads,
               float scale_log2, const __nv_bfloat16* __restrict__ q, int with_self, int prefix_len) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t smem_base = smem_u32(smem);

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int group = n_q_heads / n_kv_heads;
    const int lq = bv.q_len;
    const int rows = group * lq;
    const int rg_rows = ws.rg_rows;                                 // 256, or 128 (one row tile per CTA)
    const int row_groups = (rows + rg_rows - 1) / rg_rows;
    const int lb = blockIdx.z;                                      // layer * B + request
    const int layer = lb / bv.n_requests;
    const int b = lb - layer * bv.n_requests;
    q += (size_t)layer * q_layer_stride;
    const int kvh = blockIdx.y / row_groups;
    const int rg = blockIdx.y - kvh * row_groups;
    const int rows_here = min(rg_rows, rows - rg * rg_rows);
    const bool alternate = rows_here <= 128;                        // both warpgroups on the same rows
    const int n_qt = alternate ? 1 : 2;                             // query tiles in shared memory
    const int n_stages = kSmemTiles - n_qt;                         // 6 or 5
    const int n_parts = ws.n_splits;                                // parts per request, even
    const int pair = blockIdx.x;                                    // this CTA fills parts 2*pair, 2*pair+1
    const int rows_total = n_q_heads * lq;

    // shared memory map: [Q tiles][ring][barriers]
    const uint32_t q_base = smem_base;
    const uint32_t ring_base = q_base + n_qt * kTileBytes;
    Barriers* bars = reinterpret_cast<Barriers*>(smem + kSmemTiles * kTileBytes);
    int2* s_meta = reinterpret_cast<int2*>(smem + kSmemTiles * kTileBytes + 512);
    volatile int* abort_flag = &bars->abort_flag;

    const int tbase = pv.tile_begin[b];
    const int n_tiles = pv.n_tiles[b];
    const int n_pairs = n_parts >> 1;
    const int t_begin = (int)((long long)n_tiles * pair / n_pairs);
    const int t_end = (int)((long long)n_tiles * (pair + 1) / n_pairs);
    // the CTA of the last pair of parts also takes the prefix cache and the query-self block, as more tiles after its
    // documents'
    const bool last_pair = pair == n_pairs - 1;
    const bool has_self = with_self && last_pair;
    const int n_doc_it = t_end - t_begin;
    const int n_prefix_it = last_pair ? (prefix_len + kTile - 1) / kTile : 0;
    const int n_it = n_doc_it + n_prefix_it + (has_self ? 1 : 0);   // key tiles of this CTA
    const ExtraTiles ex = {n_doc_it, n_prefix_it, prefix_len, has_self ? n_it - 1 : -1, b * lq, lq};
    // first workspace row of this CTA in part 2*pair
    const size_t slot0 = ((size_t)lb * n_parts + 2 * pair) * rows_total + (size_t)kvh * rows + rg * rg_rows;

    // rows that will carry no data in one of the two parts: mark them neutral (m = -inf)
    for (int r = tid; r < rows_here; r += kThreads) {
        if (n_it <= 0) ws.part_m[slot0 + r] = -INFINITY;
        if (n_it <= 0 || !alternate || n_it < 2) ws.part_m[slot0 + rows_total + r] = -INFINITY;
    }
    if (n_it <= 0) return;
    const int ti0 = tbase + t_begin;                                // first tile of this CTA in the plan's list
    if (tid < min(n_doc_it, kMetaTiles)) {
        const int len = pv.tile_len[ti0 + tid], doc = pv.tile_doc[ti0 + tid];
        s_meta[tid] = make_int2(pv.tile_row0[ti0 + tid], (len & 0xff) | (doc << 8));   // len 1..128 -> 0x80 at most
    }
    // query rows of this CTA: the loads are issued now so that their latency overlaps the set-up below
    uint4 qval[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int idx = tid + i * kThreads;
        const int chunk = idx & 15, r = idx >> 4;                   // r: row within the CTA's row group
        qval[i] = make_uint4(0u, 0u, 0u, 0u);
        if (i < 4 * n_qt && r < rows_here) {
            const int row = rg * rg_rows + r;
            const int g = row / lq, j = row - g * lq;
            const int h = kvh * group + g;
            qval[i] = __ldg(reinterpret_cast<const uint4*>(q + (((size_t)b * lq + j) * n_q_heads + h) * kD + chunk * 8));
        }
    }

    if (tid == 0) {
        const int rows_t0 = min(rows_here, 128), rows_t1 = alternate ? rows_t0 : rows_here - 128;
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(smem_u32(&bars->kv_full[s][0]), 1);
            mbar_init(smem_u32(&bars->kv_full[s][1]), 1);
            mbar_init(smem_u32(&bars->kv_empty[s]), 1);
            mbar_init(smem_u32(&bars->k_ready[s]), kRotateThreads);
        }
        for (int w = 0; w < 2; ++w) {
            const int active = 32 * (((w ? rows_t1 : rows_t0) + 31) / 32);   // threads of warps that own rows
            mbar_init(smem_u32(&bars->s_full[w]), 1);
            mbar_init(smem_u32(&bars->p_ready[w]), active);
            mbar_init(smem_u32(&bars->o_done[w]), 1);
        }
        bars->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 13) {                                               // all 512 TMEM columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&bars->tmem_base)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    __syncthreads();                                                // barriers are initialised

    // the producer starts streaming before the query tile is staged
    int produced = 0;
    auto produce = [&](int u) {                                     // u-th ring use: K(u/2) if even, V(u/2) if odd
        const int st = ring_mod(u, alternate);
        const TileInfo tile = tile_info(s_meta, pv, ti0, u >> 1, ex);
        const int row0 = tile.row0;
        const int boxes = (tile.len + kBoxRows - 1) / kBoxRows;
        const CUtensorMap* map = tile.doc == -1 ? ((u & 1) ? &maps.vs[boxes - 1] : &maps.ks[boxes - 1])
                                 : tile.doc == -2 ? ((u & 1) ? &maps.vp[boxes - 1] : &maps.kp[boxes - 1])
                                                  : ((u & 1) ? &maps.v[boxes - 1] : &maps.k[boxes - 1]);
        const uint32_t bar = smem_u32(&bars->kv_full[st][u & 1]);
        const uint32_t dst = ring_base + st * kTileBytes;
        mbar_expect_tx(bar, boxes * 2 * kBoxBytes);
        tma_load_4d(dst, map, 0, kvh, row0, layer, bar);
        tma_load_4d(dst + kHalfBytes, map, 64, kvh, row0, layer, bar);
    };
    if (warp == 12 && lane == 0) {
        for (int i = 0; i < 4; ++i) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.k[i]) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.v[i]) : "memory");
        }
        for (; produced < 2; ++produced) produce(produced);        // first key and value tile; the rest follow below
    }

    // query rows into swizzled shared memory (zero rows beyond the valid ones)
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int idx = tid + i * kThreads;
        const int chunk = idx & 15, r = idx >> 4;
        if (i < 4 * n_qt) {
            const int mt = r >> 7, rr = r & 127;
            *reinterpret_cast<uint4*>(smem + (size_t)mt * kTileBytes + (chunk >> 3) * kHalfBytes + swz(rr, chunk & 7)) = qval[i];
        }
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars->tmem_base;

    // Work of warpgroup w: item j uses key tile kt(w, j) and query tile qt(w).
    //   side by side (two row tiles): kt = j,          n_items = n_it
    //   alternating  (one row tile):  kt = 2 j + w,    n_items = ceil((n_it - w) / 2)
    if (warp == 12 || warp == 13) {
        if (warp == 12 && lane == 0) {
            // -------------------------------------------------------------- TMA producer
            for (int u = produced; u < 2 * n_it; ++u) {
                const int st = ring_mod(u, alternate);
                if (u >= n_stages && !mbar_wait(smem_u32(&bars->kv_empty[st]), (ring_div(u, alternate) - 1) & 1, abort_flag)) break;
                produce(u);
            }
        } else if (warp == 13 && lane == 0) {
            // -------------------------------------------------------------- MMA issue
            // Sequence entry n: warpgroup w = n & 1, its item j = n >> 1, key tile = n (alternating)
            // or j (side by side).  Issue order: S(0) S(1), then PV(n) followed by S(n + 2): the
            // next QK^T of a warpgroup follows its own PV in the pipe, so S may overwrite the P it aliases.
            // This one thread is the pacemaker of the CTA: whatever it executes between two bursts of
            // tcgen05.mma is time in which the tensor cores idle.  Its ring positions and barrier parities are
            // therefore running counters, and every descriptor is a precomputed base plus a stage offset.
            const uint32_t idesc_o = instr_desc(kD, true);
            const uint32_t idesc_s0 = instr_desc(0, false);
            const int n_seq = alternate ? n_it : 2 * n_it;
            const int period = alternate ? 3 : 5;                   // tiles after which a stage's parity flips
            const uint64_t a_desc0 = smem_desc(q_base, 16, 1024);
            const uint64_t a_desc1 = alternate ? a_desc0 : smem_desc(q_base + kTileBytes, 16, 1024);
            const uint64_t bk_desc = smem_desc(ring_base, 16, 1024);
            const uint64_t bv_desc = smem_desc(ring_base, kHalfBytes, 1024);
            const uint32_t bar_k_ready = smem_u32(&bars->k_ready[0]), bar_kv_full = smem_u32(&bars->kv_full[0][0]);
            const uint32_t bar_kv_empty = smem_u32(&bars->kv_empty[0]);
            const uint32_t bar_s_full = smem_u32(&bars->s_full[0]), bar_p_ready = smem_u32(&bars->p_ready[0]);
            const uint32_t bar_o_done = smem_u32(&bars->o_done[0]);
            // position of the next tile of one kind (keys: stages 0, 2, 4, ...; values: 1, 3, 5, ...) in the ring
            struct Cursor {
                int stage, parity, count, tile;
            };
            auto advance = [&](Cursor& c) {
                c.stage += 2;
                if (c.stage >= n_stages) c.stage -= n_stages;
                if (++c.count == period) {
                    c.count = 0;
                    c.parity ^= 1;
                }
                ++c.tile;
            };
            auto keys_of = [&](int it) -> int {                     // MMA extent of a tile: its rows rounded up to 16
                return (tile_info(s_meta, pv, ti0, it, ex).len + 15) & ~15;
            };
            Cursor ck = {0, 0, 0, 0}, cv = {1, 0, 0, 0};            // keys for the next QK^T, values for the next PV
            auto issue_s = [&](int n) -> bool {
                const int w = n & 1;
                const int n_keys = keys_of(ck.tile);
                if (!mbar_wait(ROTATE ? bar_k_ready + ck.stage * 8 : bar_kv_full + ck.stage * 16, ck.parity, abort_flag)) return false;
                tc_fence_after();
                const uint64_t a0 = w ? a_desc1 : a_desc0;
                const uint64_t b0 = bk_desc + (uint64_t)(ck.stage * (kTileBytes >> 4));
                const uint32_t idesc_s = idesc_s0 | ((uint32_t)(n_keys >> 3) << 17);
                const uint32_t s_tmem = tmem + w * 128;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {                    // 16 dims per instruction
                    const uint64_t off = (uint64_t)(((kk >> 2) * kHalfBytes + (kk & 3) * 32) >> 4);
                    umma(s_tmem, a0 + off, b0 + off, idesc_s, kk > 0);
                }
                umma_commit(bar_s_full + w * 8);
                if (alternate || w == 1) {                          // last reader of the keys
                    umma_commit(bar_kv_empty + ck.stage * 8);
                    advance(ck);
                }
                return true;
            };
            auto issue_pv = [&](int n) -> bool {
                const int w = n & 1, j = n >> 1;
                const int n_steps = keys_of(cv.tile) >> 4;          // 16 keys = 8 packed columns per instruction
                if (!mbar_wait(bar_kv_full + cv.stage * 16 + 8, cv.parity, abort_flag)) return false;
                if (!mbar_wait(bar_p_ready + w * 8, j & 1, abort_flag)) return false;
                tc_fence_after();
                const uint64_t b0 = bv_desc + (uint64_t)(cv.stage * (kTileBytes >> 4));
                const uint32_t o_tmem = tmem + 256 + w * 128, p_tmem = tmem + w * 128;
                umma_ts(o_tmem, p_tmem, b0, idesc_o, j > 0);
#pragma unroll
                for (int kk = 1; kk < kTile / 16; ++kk)
                    if (kk < n_steps) umma_ts(o_tmem, p_tmem + kk * 8, b0 + (uint64_t)(kk * 128), idesc_o, 1u);
                umma_commit(bar_o_done + w * 8);
                if (alternate || w == 1) {                          // last reader of the values
                    umma_commit(bar_kv_empty + cv.stage * 8);
                    advance(cv);
                }
                return true;
            };
            bool ok = issue_s(0);
            if (ok && n_seq > 1) ok = issue_s(1);
            for (int n = 0; n < n_seq && ok; ++n) {
                ok = issue_pv(n);
                if (ok && n + 2 < n_seq) ok = issue_s(n + 2);
            }
        }
    } else if (warp >= 8 && !ROTATE) {
        // keys are used as cached: nothing to do
    } else if (warp >= 8) {
        // ------------------------------------------------------------------ key rotation (Eq. 5)
        const int t = warp < 12 ? tid - 256 : tid - 320;            // 0..191 (warps 8-11, 14, 15)
        const int chunk = t & 7, rsub = t >> 3;
        for (int it = 0; it < n_it; ++it) {
            const TileInfo tile = tile_info(s_meta, pv, ti0, it, ex);
            const int len = tile.len;
            const float2* trig = pv.trig + (size_t)max(tile.doc, 0) * (kD / 2);
            const int st = ring_mod(2 * it, alternate);
            float2 cs[8];
            if (tile.doc < 0) {                                     // the query's own keys are already in place
#pragma unroll
                for (int e = 0; e < 8; ++e) cs[e] = make_float2(1.f, 0.f);
            } else if (LAYOUT == CF_ROPE_HALF) {
#pragma unroll
                for (int e = 0; e < 8; ++e) cs[e] = __ldg(trig + chunk * 8 + e);
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    cs[e] = __ldg(trig + chunk * 4 + e);            // first half: dims chunk*8 .. +7
                    cs[4 + e] = __ldg(trig + 32 + chunk * 4 + e);   // second half: dims 64 + chunk*8 ..
                }
            }
            const int kuse = ring_uses(it, alternate);                        // key loads this stage has seen
            if (!mbar_wait(smem_u32(&bars->kv_full[st][0]), kuse & 1, abort_flag)) break;
            unsigned char* buf = smem + (ring_base - smem_base) + (size_t)st * kTileBytes;
#pragma unroll 2
            for (int r = rsub; r < len; r += kRotateThreads / 8) {
                uint4* pa = reinterpret_cast<uint4*>(buf + swz(r, chunk));
                uint4* pb = reinterpret_cast<uint4*>(buf + kHalfBytes + swz(r, chunk));
                uint4 va = *pa, vb = *pb;
                uint32_t wa[4] = {va.x, va.y, va.z, va.w}, wb[4] = {vb.x, vb.y, vb.z, vb.w};
                if (LAYOUT == CF_ROPE_HALF) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        float a0 = __uint_as_float(wa[i] << 16), a1 = __uint_as_float(wa[i] & 0xffff0000u);
                        float b0 = __uint_as_float(wb[i] << 16), b1 = __uint_as_float(wb[i] & 0xffff0000u);
                        float ya0, yb0, ya1, yb1;
                        rotate_pair(a0, b0, cs[2 * i].x, cs[2 * i].y, ya0, yb0);
                        rotate_pair(a1, b1, cs[2 * i + 1].x, cs[2 * i + 1].y, ya1, yb1);
                        wa[i] = pack_bf16(ya0, ya1);
                        wb[i] = pack_bf16(yb0, yb1);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        float a0 = __uint_as_float(wa[i] << 16), a1 = __uint_as_float(wa[i] & 0xffff0000u);
                        float b0 = __uint_as_float(wb[i] << 16), b1 = __uint_as_float(wb[i] & 0xffff0000u);
                        float ya0, ya1, yb0, yb1;
                        rotate_pair(a0, a1, cs[i].x, cs[i].y, ya0, ya1);
                        rotate_pair(b0, b1, cs[4 + i].x, cs[4 + i].y, yb0, yb1);
                        wa[i] = pack_bf16(ya0, ya1);
                        wb[i] = pack_bf16(yb0, yb1);
                    }
                }
                *pa = make_uint4(wa[0], wa[1], wa[2], wa[3]);
                *pb = make_uint4(wb[0], wb[1], wb[2], wb[3]);
            }
            fence_proxy_async();
            mbar_arrive(smem_u32(&bars->k_ready[st]));
        }
    } else {
        // ------------------------------------------------------------------ softmax, one row per thread
        const int w = warp >> 2;                                    // warpgroup
        const int r = tid & 127;                                    // row within the tile = TMEM lane
        const int row_in_group = (alternate ? 0 : w * 128) + r;
        const int n_items = alternate ? (n_it - w + 1) / 2 : n_it;
        // a warp none of whose rows exist does not take part (the barrier counts exclude it)
        const bool warp_active = (alternate ? 0 : w * 128) + (warp & 3) * 32 < rows_here;
        if (warp_active && n_items > 0) {
            const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
            const uint32_t s_addr = tmem + lane_addr + w * 128;
            const uint32_t o_addr = tmem + lane_addr + 256 + w * 128;
            const bool row_valid = row_in_group < rows_here;
            const size_t tile_row = (size_t)kvh * rows + rg * rg_rows + row_in_group;
            float* tile_lse2 = ws.tile_lse2 + (size_t)layer * ws.max_tiles * rows_total;
            float m_ref = -INFINITY, l_run = 0.f, l_docs = 0.f;     // l_docs: the sum over the documents' keys alone
            bool seen_extra = false;
            const int q_index = (rg * rg_rows + row_in_group) % lq;     // position of this row's token in the query
            bool ok = true;
            for (int j = 0; j < n_items; ++j) {
                const int it = alternate ? 2 * j + w : j;
                const int ti = ti0 + it;
                const int len = tile_info(s_meta, pv, ti0, it, ex).len;
                // keys this row may see: the whole tile of a document, the query tokens 0..q_index of the
                // query-self block (causal mask, footnote to Eq. 1)
                const int vis = it == ex.self_it ? min(len, q_index + 1) : len;
                if (it >= ex.first && !seen_extra) {                // from here on the keys are not the documents'
                    l_docs = l_run;
                    seen_extra = true;
                }
                ok = mbar_wait(smem_u32(&bars->s_full[w]), j & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                if (j > 0) {
                    // PV(j-1) sits before S(j) in the tensor pipe, so it is complete; waiting here keeps
                    // this thread's view of the barrier in step (every phase is waited for, in order)
                    ok = mbar_wait(smem_u32(&bars->o_done[w]), (j - 1) & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                }
                // Single pass over S in 32-key chunks, loads double-buffered.  The reference maximum only
                // moves when a chunk exceeds it by more than 2^8; then O, the sums and the P chunks of this
                // tile that are already written are rescaled (rare after the first chunk of the first tile).
                const int n_chunks = (len + 31) >> 5;
                float tile_sum = 0.f;
                uint32_t va[32], vb[32];
                // step 1 of a chunk; no tensor-memory load may be in flight across these branches
                auto prepare = [&](const uint32_t (&v)[32], int valid, int c) {
                    const float cmax = (valid >= 32 ? chunk_max<false>(v, 32) : chunk_max<true>(v, valid)) * scale_log2;
                    const bool move = cmax > m_ref + kRescaleThreshold;       // very first chunk: m_ref = -inf
                    if (__any_sync(0xffffffffu, move)) {
                        float alpha = 1.f;
                        if (move) {
                            alpha = fast_exp2(m_ref - cmax);                  // 0 when nothing is accumulated yet
                            m_ref = cmax;
                        }
                        if (j > 0) {
                            for (int cc = 0; cc < 8; ++cc) {
                                uint32_t o[16];
                                tmem_ld16(o_addr + cc * 16, o);
#pragma unroll
                                for (int k = 0; k < 16; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * alpha);
                                tmem_st16(o_addr + cc * 16, o);
                            }
                        }
                        if (c > 0) asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");   // P stores in flight
                        for (int cc = 0; cc < c; ++cc) {
                            uint32_t pk[16];
                            tmem_ld16(s_addr + cc * 16, pk);
#pragma unroll
                            for (int k = 0; k < 16; ++k)
                                pk[k] = pack_bf16(__uint_as_float(pk[k] << 16) * alpha, __uint_as_float(pk[k] & 0xffff0000u) * alpha);
                            tmem_st16(s_addr + cc * 16, pk);
                        }
                        l_run *= alpha;
                        l_docs *= alpha;
                        tile_sum *= alpha;
                    }
                };
                // step 2 (straight-line): exponentials, packing; P chunk c lands in S columns 16c..16c+15,
                // which belong to S chunks already held in registers
                auto finish = [&](uint32_t (&v)[32], int valid, int c) {
                    tile_sum += valid >= 32 ? chunk_exp<false>(v, 32, scale_log2, -m_ref) : chunk_exp<true>(v, valid, scale_log2, -m_ref);
                    tmem_st16_async(s_addr + c * 16, v);
                };
                tmem_ld32_async(s_addr, va);
                tmem_ld_wait(va);
                for (int c = 0; c < n_chunks; c += 2) {
                    prepare(va, vis - c * 32, c);
                    if (c + 1 < n_chunks) tmem_ld32_async(s_addr + (c + 1) * 32, vb);
                    finish(va, vis - c * 32, c);
                    if (c + 1 < n_chunks) {
                        tmem_ld_wait(vb);
                        prepare(vb, vis - c * 32 - 32, c + 1);
                        if (c + 2 < n_chunks) tmem_ld32_async(s_addr + (c + 2) * 32, va);
                        finish(vb, vis - c * 32 - 32, c + 1);
                        if (c + 2 < n_chunks) tmem_ld_wait(va);
                    }
                }
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                tc_fence_before();
                mbar_arrive(smem_u32(&bars->p_ready[w]));
                if (it < ex.first && row_valid) tile_lse2[(size_t)ti * rows_total + tile_row] = m_ref + log2f(tile_sum);
                l_run += tile_sum;
            }
            if (ok) ok = mbar_wait(smem_u32(&bars->o_done[w]), (n_items - 1) & 1, abort_flag);
            if (ok) {
                tc_fence_after();
                const size_t slot = slot0 + (alternate ? (size_t)w * rows_total : 0) + row_in_group;
                // Partial O rows leave as bf16 through shared memory so that global stores are full
                // 256-byte rows.  Staging space: this warpgroup's own query tile (every QK^T that read
                // it has completed), or, when both warpgroups share one query tile, the ring stage of
                // the next unused key or value slot (its last reader completed before this point).
                unsigned char* stage = alternate ? smem + (ring_base - smem_base) + (size_t)((2 * n_it + w) % n_stages) * kTileBytes
                                                 : smem + (size_t)w * kTileBytes;
                for (int c = 0; c < 4; ++c) {
                    uint32_t o[32];
                    tmem_ld32(o_addr + c * 32, o);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {                   // 8 dims = one 16-byte chunk
                        const int chunk = c * 4 + i;
                        *reinterpret_cast<uint4*>(stage + r * 256 + ((chunk ^ (r & 15)) << 4)) =
                            make_uint4(pack_bf16(__uint_as_float(o[8 * i]), __uint_as_float(o[8 * i + 1])),
                                       pack_bf16(__uint_as_float(o[8 * i + 2]), __uint_as_float(o[8 * i + 3])),
                                       pack_bf16(__uint_as_float(o[8 * i + 4]), __uint_as_float(o[8 * i + 5])),
                                       pack_bf16(__uint_as_float(o[8 * i + 6]), __uint_as_float(o[8 * i + 7])));
                    }
                }
                __syncwarp();
                {
                    const int warp_row0 = r & ~31;                  // this warp's 32 rows
                    const int rows_left = rows_here - ((alternate ? 0 : w * 128) + warp_row0);
                    unsigned char* dst = reinterpret_cast<unsigned char*>(ws.part_o) + (slot - lane) * (size_t)(kD * 2);
#pragma unroll 4
                    for (int i = 0; i < 16; ++i) {                  // two rows per step, 16 lanes each
                        const int rr = 2 * i + (lane >> 4), chunk = lane & 15;
                        if (rr < rows_left) {
                            const int srow = warp_row0 + rr;
                            const uint4 val = *reinterpret_cast<const uint4*>(stage + srow * 256 + ((chunk ^ (srow & 15)) << 4));
                            *reinterpret_cast<uint4*>(dst + (size_t)rr * (kD * 2) + chunk * 16) = val;
                        }
                    }
                }
                if (row_valid) {
                    ws.part_m[slot] = m_ref;
                    ws.part_l[slot] = l_run;
                    // this part's sum over the documents alone: what the document scores are measured against
                    if (ws.part_ld) ws.part_ld[slot] = seen_extra ? l_docs : l_run;
                }
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (bars->abort_flag) {
        // a wait expired: let loads already in flight land before the shared memory is given back
        if (warp == 12 && lane == 0) {
            for (int u = 0; u < 2 * n_it; ++u) {
                const int use = (n_stages & 1) ? (u >> 1) / n_stages : u / n_stages;
                const uint32_t bar = smem_u32(&bars->kv_full[u % n_stages][u & 1]);
                const long long t0 = clock64();
                while (!mbar_try_wait(bar, use & 1) && clock64() - t0 < kWaitLimitCycles / 16) {}
            }
        }
        if (tid == 0) atomicCAS(pv.status, 0, CF_ERR_TIMEOUT);
        __syncthreads();
    }
    if (warp == 13) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
    }
}

// Exercises the bounded wait by itself: one CTA initialises an mbarrier that nothing ever arrives on,
// every thread waits on it with the given limit, the wait gives up, and the CTA reports
// CF_ERR_TIMEOUT through the status word exactly as the attention kernel does.  No tensor memory,
// no copies in flight: the kernel returns by itself after about `limit_cycles` clocks.
__global__ void __launch_bounds__(128) wait_probe_kernel(int* status, long long limit_cycles) {
    __shared__ unsigned long long bar;
    __shared__ int abort_word;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const bool ok = mbar_wait(smem_u32(&bar), 0, &abort_word, limit_cycles);
    __syncthreads();
    if (threadIdx.x == 0 && !ok && abort_word) atomicCAS(status, 0, CF_ERR_TIMEOUT);
}

// The store as a 4-D tensor (head_dim, kv heads, rows, layers).
int make_store_map(CUtensorMap* map, const void* base, const cf_geom* g, const cf_batch* b, const LayerSpan& span,
                   int box_rows) {
    const unsigned long long layer_bytes = span.n_layers > 1 ? (unsigned long long)span.kv_stride * 2
                                                             : (unsigned long long)b->total_tokens * b->token_stride * 2;
    return make_rows_map(map, base, g->n_kv_heads, (unsigned long long)b->total_tokens,
                         (unsigned long long)b->token_stride * 2, span.n_layers, layer_bytes, box_rows);
}

// Keys or values of the query tokens, [layers][requests][q_len][kv heads][head_dim], as a 4-D tensor
// (head_dim, kv heads, requests * q_len rows, layers).
int make_self_map(CUtensorMap* map, const void* base, const cf_geom* g, const cf_batch* b, const LayerSpan& span,
                  long long self_stride, int box_rows) {
    const unsigned long long rows = (unsigned long long)b->n_requests * b->q_len;
    const unsigned long long row_bytes = (unsigned long long)g->n_kv_heads * kD * 2;
    const unsigned long long layer_bytes = span.n_layers > 1 ? (unsigned long long)self_stride * 2 : rows * row_bytes;
    return make_rows_map(map, base, g->n_kv_heads, rows, row_bytes, span.n_layers, layer_bytes, box_rows);
}

// Keys or values of a shared prefix cache, [layers][prefix_len][kv heads][head_dim] dense, as a 4-D tensor
// (head_dim, kv heads, prefix rows, layers).
int make_prefix_map(CUtensorMap* map, const void* base, const cf_geom* g, const LayerSpan& span, int prefix_len,
                    long long prefix_stride, int box_rows) {
    const unsigned long long row_bytes = (unsigned long long)g->n_kv_heads * kD * 2;
    const unsigned long long layer_bytes = span.n_layers > 1 ? (unsigned long long)prefix_stride * 2
                                                             : (unsigned long long)prefix_len * row_bytes;
    return make_rows_map(map, base, g->n_kv_heads, (unsigned long long)prefix_len, row_bytes, span.n_layers, layer_bytes, box_rows);
}

}  // namespace

int launch_wait_probe(const PlanView& pv, long long limit_cycles, cudaStream_t stream) {
    wait_probe_kernel<<<1, 128, 0, stream>>>(pv.status, limit_cycles);
    return cudaGetLastError() == cudaSuccess ? CF_OK : CF_ERR_CUDA;
}

bool attn_tc_supported(const cf_geom* g, const cf_batch* b) {
    return g->dtype == CF_BF16 && g->head_dim == 128 && b->total_tokens > 0 && b->n_docs_total < (1 << 23);
}

int launch_attn_tc(const cf_geom* g, const cf_batch* b, const PlanView& pv, const LayerSpan& span, const void* q,
                   const void* k, const void* v, const void* k_self, const void* v_self, long long self_stride,
                   const void* k_prefix, const void* v_prefix, long long prefix_stride, int prefix_len,
                   float scale_log2, const AttnWorkspace& ws, cudaStream_t stream) {
    const int rows = (g->n_q_heads / g->n_kv_heads) * b->q_len;
    const int row_groups = (rows + ws.rg_rows - 1) / ws.rg_rows;
    if ((long long)g->n_kv_heads * row_groups > 65535 || (long long)b->n_requests * span.n_layers > 65535 ||
        (ws.n_splits & 1) || (ws.rg_rows != 128 && ws.rg_rows != 256))
        return CF_ERR_INVALID_ARG;
    StoreMaps maps;
    for (int i = 0; i < 4; ++i) {
        int rc = make_store_map(&maps.k[i], k, g, b, span, (i + 1) * kBoxRows);
        if (rc != CF_OK) return rc;
        rc = make_store_map(&maps.v[i], v, g, b, span, (i + 1) * kBoxRows);
        if (rc != CF_OK) return rc;
        if (k_self) {
            rc = make_self_map(&maps.ks[i], k_self, g, b, span, self_stride, (i + 1) * kBoxRows);
            if (rc != CF_OK) return rc;
            rc = make_self_map(&maps.vs[i], v_self, g, b, span, self_stride, (i + 1) * kBoxRows);
            if (rc != CF_OK) return rc;
        } else {
            maps.ks[i] = maps.k[i];
            maps.vs[i] = maps.v[i];
        }
        if (prefix_len > 0) {
            rc = make_prefix_map(&maps.kp[i], k_prefix, g, span, prefix_len, prefix_stride, (i + 1) * kBoxRows);
            if (rc != CF_OK) return rc;
            rc = make_prefix_map(&maps.vp[i], v_prefix, g, span, prefix_len, prefix_stride, (i + 1) * kBoxRows);
            if (rc != CF_OK) return rc;
        } else {
            maps.kp[i] = maps.k[i];
            maps.vp[i] = maps.v[i];
        }
    }
    if (k_self && b->q_len > kTile) return CF_ERR_UNSUPPORTED;   // the query-self block is one key tile
    dim3 grid((unsigned)(ws.n_splits / 2), (unsigned)(g->n_kv_heads * row_groups),
              (unsigned)(b->n_requests * span.n_layers));
    BatchView bv = make_batch_view(b);
    static PerDeviceOnce configured[3];
    auto run = [&](auto kernel, int which) {
        if (configure_smem_once(configured[which], kernel, kSmemBytes) != CF_OK) return CF_ERR_CUDA;
        kernel<<<grid, kThreads, kSmemBytes, stream>>>(maps, bv, pv, ws, span.q_stride, g->n_q_heads,
                                                       g->n_kv_heads, scale_log2, static_cast<const __nv_bfloat16*>(q),
                                                       k_self ? 1 : 0, prefix_len);
        return cudaGetLastError() == cudaSuccess ? CF_OK : CF_ERR_CUDA;
    };
    if (ws.keys_in_place) return run(attn_tc_kernel<CF_ROPE_HALF, false>, 2);      // the slice layout plays no part
    if (g->rope_layout == CF_ROPE_HALF) return run(attn_tc_kernel<CF_ROPE_HALF, true>, 0);
    return run(attn_tc_kernel<CF_ROPE_INTERLEAVED, true>, 1);
}

}  // namespace cf
