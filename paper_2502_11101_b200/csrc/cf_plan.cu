// Device-side bookkeeping of a request batch: the kept list and its order (Algorithm 2:
// Init, argsort of S, prun), the positional allocation of the kept documents (Sec. 2.3.1 Eq. 6,
// Sec. 2.5), and what the hot kernels consume: per-document rotation tables (Eq. 2 angles of
// the delta of Eq. 5) and the list of key tiles.  One thread block per request; everything
// runs in stream order so a layer stack needs no host round trip between layers.
#include <algorithm>
#include <cmath>

#include "cf_common.cuh"

namespace cf {

constexpr int kPlanThreads = 1024;
static_assert(kPlanThreads >= kMaxDocs, "every rank of a request has a thread of its own");

__device__ __forceinline__ void raise_status(int* status, int code) { atomicCAS(status, 0, code); }

// Rotary frequencies theta^(-2p/D), p < D/2 (Eq. 2), computed once on the host: in fp64, and as
// a fraction of a full turn in units of 2^-64 (frequency / 2 pi), which lets the device reduce
// position * frequency modulo one turn in exact 64-bit integer arithmetic.
struct InvFreq {
    double f[64];
    unsigned long long turns[64];
};

// cos and sin of an fp64 angle to about 2e-9 absolute, for |x| up to ~1e5 (positions times a
// frequency <= 1): two-step Cody-Waite reduction by pi/2, then the Taylor polynomials of sin and
// cos on [-pi/4, pi/4] (remainders x^11/11! < 2e-9 and x^12/12! < 2e-10).  Used for fp32 caches,
// whose rotated keys are held to a few fp32 ulp.
__device__ __forceinline__ void sincos_reduced(double x, double& sn, double& cs) {
    const double n = rint(x * 0.63661977236758134308);               // 2/pi
    double r = fma(-n, 1.57079632679489655800e+00, x);               // pi/2, high part
    r = fma(-n, 6.12323399573676603587e-17, r);                      // pi/2, low part
    const double r2 = r * r;
    double ps = fma(r2, 2.75573192239858906526e-06, -1.98412698412698412698e-04);   // 1/9!, -1/7!
    ps = fma(ps, r2, 8.33333333333333333333e-03);                    // 1/5!
    ps = fma(ps, r2, -1.66666666666666666667e-01);                   // -1/3!
    ps = fma(ps * r2, r, r);
    double pc = fma(r2, -2.75573192239858906526e-07, 2.48015873015873015873e-05);   // -1/10!, 1/8!
    pc = fma(pc, r2, -1.38888888888888888889e-03);                   // -1/6!
    pc = fma(pc, r2, 4.16666666666666666667e-02);                    // 1/4!
    pc = fma(pc, r2, -0.5);
    pc = fma(pc, r2, 1.0);
    const int q = (int)((long long)n & 3);                           // quadrant (two's complement: works for n < 0)
    const double s0 = (q & 1) ? pc : ps, c0 = (q & 1) ? ps : pc;
    sn = (q & 2) ? -s0 : s0;
    cs = ((q + 1) & 2) ? -c0 : c0;
}

// cos and sin of delta positions at a frequency given in 2^-64 turns: the phase modulo one turn is
// an exact wrapping 64-bit product, split into the nearest quarter turn and a remainder r in
// [-pi/4, pi/4).  r is carried as a pair of floats (r_hi + r_lo, about 48 bits), and the Taylor
// polynomials add their small terms to r_hi (sin) and to 1 (cos) last, so the results are within
// about 7e-8 of the exact values -- fp32 tables for bf16 caches (bf16 spacing is 4e-3) without
// any fp64 arithmetic.
__device__ __forceinline__ void sincos_turns(int delta, unsigned long long turns, float& sn, float& cs) {
    const unsigned long long phase = (unsigned long long)(long long)delta * turns;
    const unsigned long long quarter = (phase + (1ull << 61)) >> 62;                 // nearest quarter turn, 0..3
    const long long rem = (long long)(phase - (quarter << 62));                      // [-2^61, 2^61) of 2^-64 turns
    const float top = (float)(int)(rem >> 37);                                       // 25 signed bits, units of 2^-27 turn
    const float low = (float)(int)((rem >> 13) & 0xFFFFFF);                          // the next 24 bits
    constexpr double kStep = 6.283185307179586476925 / 134217728.0;                  // 2 pi / 2^27
    constexpr float kStepHi = (float)kStep;
    constexpr float kStepLo = (float)(kStep - (double)kStepHi);
    constexpr float kStepLow = (float)(kStep / 16777216.0);
    const float r_hi = top * kStepHi;
    const float r_lo = fmaf(top, kStepLo, fmaf(top, kStepHi, -r_hi)) + low * kStepLow;
    const float r2 = r_hi * r_hi;
    float ps = fmaf(r2, 2.7557319e-6f, -1.9841270e-4f);                              // 1/9!, -1/7!
    ps = fmaf(ps, r2, 8.3333333e-3f);                                                // 1/5!
    ps = fmaf(ps, r2, -1.6666667e-1f);                                               // -1/3!
    const float s0 = r_hi + fmaf(ps * r2, r_hi, r_lo);
    float pc = fmaf(r2, -2.7557319e-7f, 2.4801587e-5f);                              // -1/10!, 1/8!
    pc = fmaf(pc, r2, -1.3888889e-3f);                                               // -1/6!
    pc = fmaf(pc, r2, 4.1666667e-2f);                                                // 1/4!
    pc = fmaf(pc, r2, -0.5f);
    const float c0 = 1.0f + fmaf(pc, r2, -(r_hi * r_lo));
    const int q = (int)quarter;
    const float s1 = (q & 1) ? c0 : s0, c1 = (q & 1) ? s0 : c0;
    sn = (q & 2) ? -s1 : s1;
    cs = ((q + 1) & 2) ? -c1 : c1;
}

// Exclusive prefix sum of one value per thread over the block; *total receives the sum.  Every
// thread of the block must call it.
__device__ __forceinline__ int block_scan(int value, int* s_warp_sum, int* total) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int incl = value;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) s_warp_sum[warp] = incl;
    __syncthreads();
    if (warp == 0) {                                     // scan of the (at most 32) warp sums
        const int mine = lane < (int)(blockDim.x >> 5) ? s_warp_sum[lane] : 0;
        int acc = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, acc, o);
            if (lane >= o) acc += up;
        }
        s_warp_sum[lane] = acc - mine;                   // sum of the warps before this one
        if (lane == 31) s_warp_sum[32] = acc;
    }
    __syncthreads();
    const int before = s_warp_sum[warp] + incl - value;
    *total = s_warp_sum[32];
    __syncthreads();
    return before;
}

// mode 0: initialise from (order, kept_count); mode 1: prune by score, then rebuild.
// Everything a later step needs from global memory is staged in shared memory at the start, the
// serial steps of the method (ranking, walking a window backwards from the query, numbering the
// tiles) are written as counting and prefix sums over the whole block, and the results leave for
// global memory together at the end: no barrier in between has stores in flight to wait for.
__global__ void __launch_bounds__(kPlanThreads)
plan_kernel(GeomView gv, BatchView bv, PlanView pv, InvFreq inv_freq, int mode, const int* __restrict__ order,
            const int* __restrict__ kept_count_in, int query_start_arg,
            const float* __restrict__ score_accum, int keep, const int* __restrict__ keep_per_request,
            int strategy) {
    __shared__ int s_ids[kMaxDocs];       // kept local ids by rank
    __shared__ int s_tmp[kMaxDocs];       // new order; running lengths of the windows; first tile of every rank
    __shared__ int s_row[kMaxDocs + 1];   // first store row of every document (by local id), and the end
    __shared__ int s_dst[kMaxDocs];       // start positions by local id
    __shared__ int s_group[kMaxDocs];     // window index by local id
    __shared__ int s_first[kMaxDocs];      // first tile by local id
    __shared__ int s_cnt[kMaxDocs];       // tile count by local id
    __shared__ int s_src[kMaxDocs];       // positions the documents were cached at, by local id
    __shared__ float s_score[kMaxDocs];
    __shared__ float s_all[kMaxDocs];     // accumulated scores of all documents of the request, by local id
    __shared__ unsigned char s_flag[kMaxDocs];
    __shared__ int s_longest, s_min_cursor;
    __shared__ int s_warp_sum[kPlanThreads / 32 + 1];

    const int b = blockIdx.x;
    const int tid = threadIdx.x;
    const int nthreads = (int)blockDim.x;               // at least the documents of any request, a multiple of 32
    const int doc0 = bv.req_doc_begin[b];
    const int n_docs = bv.req_doc_begin[b + 1] - doc0;
    if (n_docs > kMaxDocs || n_docs < 0) {
        if (tid == 0) {
            raise_status(pv.status, CF_ERR_INVALID_ARG);
            pv.kept_count[b] = 0;
            pv.n_tiles[b] = 0;
            pv.tile_begin[b] = 0;
        }
        return;
    }
    const int half = gv.head_dim / 2;
    const int half_log2 = half == 64 ? 6 : 5;

    // ---- stage the inputs (everything here depends on doc0 alone: one round trip to global memory) ----
    int n_old = 0, keep_b = 0, n_kept = 0;
    const int kept_count_old = mode == 0 ? 0 : pv.kept_count[b];
    const int keep_arg = (mode != 0 && keep_per_request) ? keep_per_request[b] : keep;
    const int kept_raw = (mode != 0 && tid < n_docs) ? pv.kept[doc0 + tid] : 0;    // rank tid, if there is one
    if (mode != 0 && tid < n_docs) s_all[tid] = score_accum[doc0 + tid];            // S of every document, by local id
    for (int i = tid; i <= n_docs; i += nthreads) s_row[i] = bv.doc_offsets[doc0 + i];
    for (int i = tid; i < n_docs; i += nthreads) {
        s_src[i] = bv.doc_src_start[doc0 + i];
        s_dst[i] = mode == 0 ? -1 : pv.dst_start[doc0 + i];
        s_group[i] = mode == 0 ? -1 : pv.group[doc0 + i];
    }
    int query_start = mode == 0 ? (query_start_arg < 0 ? gv.pos_range - bv.tail_reserve : query_start_arg)
                                : pv.query_start[b];
    int windows = mode == 0 ? max(1, bv.n_reuse) : pv.n_reuse[b];
    if (mode == 0) {
        n_kept = kept_count_in ? kept_count_in[b] : n_docs;
        n_kept = max(0, min(n_kept, n_docs));
        for (int i = tid; i < n_docs; i += nthreads) s_cnt[i] = 0;
        __syncthreads();
        for (int r = tid; r < n_kept; r += nthreads) {
            int id = order ? order[doc0 + r] : r;
            if (id < 0 || id >= n_docs) {
                raise_status(pv.status, CF_ERR_INVALID_ARG);
                id = 0;
            }
            if (atomicAdd(&s_cnt[id], 1) != 0) raise_status(pv.status, CF_ERR_INVALID_ARG);   // an id listed twice
            s_ids[r] = id;
        }
    } else {
        n_old = max(0, min(kept_count_old, n_docs));
        keep_b = max(0, min(keep_arg, n_old));
        if (tid < n_old) s_ids[tid] = max(0, min(kept_raw, n_docs - 1));
    }
    if (tid == 0) {
        s_longest = 0;
        s_min_cursor = 0x7fffffff;
    }
    __syncthreads();

    // ---- the kept list, in rank order -------------------------------------------------------
    if (mode != 0) {
        if (tid < n_old) s_score[tid] = s_all[s_ids[tid]];
        __syncthreads();
        // rank by counting: how many kept documents beat this one (ties: lower id wins); eight
        // lanes share the count of one document
        for (int r0 = 0; r0 < n_old; r0 += nthreads / 8) {
            const int r = r0 + (tid >> 3);
            const float sc = r < n_old ? s_score[r] : 0.f;
            const int id = r < n_old ? s_ids[r] : 0;
            int better = 0;
            if (r < n_old)
                for (int o = tid & 7; o < n_old; o += 8) {
                    const float so = s_score[o];
                    better += (so > sc) || (so == sc && s_ids[o] < id);
                }
            better += __shfl_xor_sync(0xffffffffu, better, 1);
            better += __shfl_xor_sync(0xffffffffu, better, 2);
            better += __shfl_xor_sync(0xffffffffu, better, 4);
            if (r < n_old && (tid & 7) == 0) {
                s_flag[r] = better < keep_b;
                if (strategy == CF_ALLOC_SORT && better < keep_b) s_tmp[better] = id;
            }
        }
        __syncthreads();
        if (strategy != CF_ALLOC_SORT) {                  // survivors keep their order: slot = survivors before
            const int survives = tid < n_old ? (int)s_flag[tid] : 0;
            int n_survive;
            const int before = block_scan(survives, s_warp_sum, &n_survive);
            if (survives) s_tmp[before] = s_ids[tid];
        }
        __syncthreads();
        n_kept = keep_b;
        // (the clamp only matters for malformed input -- duplicate ids, NaN scores -- where two
        //  documents can claim one slot and leave another unwritten)
        for (int r = tid; r < n_kept; r += nthreads) s_ids[r] = max(0, min(s_tmp[r], n_docs - 1));
        __syncthreads();
    }

    // ---- documents that are not kept ----------------------------------------------------------
    const bool reallocate = (mode == 0) || (strategy != CF_ALLOC_NONE);
    for (int i = tid; i < n_docs; i += nthreads) s_flag[i] = 0;
    __syncthreads();
    for (int r = tid; r < n_kept; r += nthreads) s_flag[s_ids[r]] = 1;
    __syncthreads();

    // ---- positional allocation ----------------------------------------------------------------
    if (reallocate && n_kept > 0) {
        int longest = 0;
        for (int r = tid; r < n_kept; r += nthreads) longest = max(longest, s_row[s_ids[r] + 1] - s_row[s_ids[r]]);
        atomicMax(&s_longest, longest);
        __syncthreads();
        longest = s_longest;
        const int capacity = gv.pos_range - bv.prefix_len - bv.tail_reserve;
        windows = bv.n_reuse;
        if (windows <= 0) {
            const int per_window = longest > 0 ? capacity / longest : 0;     // L / l_C of Eq. 6
            if (per_window <= 0) {
                if (tid == 0) raise_status(pv.status, CF_ERR_RANGE);
                windows = n_kept;
            } else {
                windows = (n_kept + per_window - 1) / per_window;
            }
        }
        // Window w holds the ranks w, w + windows, ... and is filled backwards from the query.  With
        // the ranks listed window by window (index x), a document starts at the query start minus the
        // lengths of its window up to and including itself: one prefix sum over x.
        const int w_used = min(windows, n_kept);
        const int small = n_kept / w_used, extra = n_kept - small * w_used;   // the first `extra` windows hold small + 1
        const int x = tid;
        int len = 0, rank = -1, first = 0;
        if (x < n_kept) {
            int w, slot;
            if (x < extra * (small + 1)) {
                w = x / (small + 1);
                slot = x - w * (small + 1);
            } else {
                const int y = x - extra * (small + 1);
                w = extra + y / small;
                slot = y - (w - extra) * small;
            }
            rank = slot * windows + w;
            first = x - slot;                                               // index of the window's first rank
            const int id = s_ids[rank];
            len = s_row[id + 1] - s_row[id];
        }
        int all_rows;
        const int before = block_scan(len, s_warp_sum, &all_rows);
        if (rank >= 0) s_tmp[x] = before;
        __syncthreads();
        int lowest = 0x7fffffff;
        if (rank >= 0) {
            const int id = s_ids[rank];
            const int start = query_start - (before - s_tmp[first] + len);
            s_dst[id] = start;
            s_group[id] = rank % windows;
            lowest = start;
        }
        atomicMin(&s_min_cursor, lowest);
        __syncthreads();
        if (tid == 0 && (s_min_cursor < bv.prefix_len || query_start + bv.tail_reserve > gv.pos_range))
            raise_status(pv.status, CF_ERR_RANGE);
    }

    // ---- key tiles: runs of at most kTile rows that never straddle two documents -----------------
    const int my_tiles = tid < n_kept ? (s_row[s_ids[tid] + 1] - s_row[s_ids[tid]] + kTile - 1) / kTile : 0;
    int total;
    const int first_tile = block_scan(my_tiles, s_warp_sum, &total);
    const int base = tile_base(doc0, s_row[0]);
    const bool fail = base + total > pv.max_tiles;       // cannot happen with a plan sized by cf_plan_layout_of

    // ---- results to global memory ---------------------------------------------------------------
    if (tid == 0) {
        if (fail) raise_status(pv.status, CF_ERR_WORKSPACE);
        pv.n_tiles[b] = fail ? 0 : total;
        pv.kept_count[b] = fail ? 0 : n_kept;
        pv.tile_begin[b] = base;
        pv.n_reuse[b] = windows;
        pv.query_start[b] = query_start;
    }
    if (fail) return;
    // every array is written with consecutive threads on consecutive elements: per-document fields
    // by document, the kept list by rank, the tile list by tile
    if (tid < n_kept) {
        s_tmp[tid] = first_tile;                             // first tile of rank tid (ascending)
        s_score[tid] = __int_as_float(my_tiles);
    }
    __syncthreads();
    if (tid < n_kept) {                                      // per-document view of the same numbers
        const int id = s_ids[tid];
        s_first[id] = first_tile;
        s_cnt[id] = my_tiles;
    }
    __syncthreads();
    for (int i = tid; i < n_docs; i += nthreads) {
        const bool kept = s_flag[i] != 0;
        pv.dst_start[doc0 + i] = kept ? s_dst[i] : -1;
        pv.group[doc0 + i] = kept ? s_group[i] : -1;
        pv.doc_tile_begin[doc0 + i] = kept ? base + s_first[i] : 0;
        pv.doc_tile_count[doc0 + i] = kept ? s_cnt[i] : 0;
    }
    if (tid < n_kept) pv.kept[doc0 + tid] = s_ids[tid];
    for (int x = tid; x < total; x += nthreads) {
        int lo = 0, hi = n_kept;                             // last rank whose first tile is <= x
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_tmp[mid] <= x) lo = mid; else hi = mid;
        }
        const int id = s_ids[lo];
        const int row0 = s_row[id];
        const int len = s_row[id + 1] - row0;
        const int count = __float_as_int(s_score[lo]);
        const int t = x - s_tmp[lo];
        // the document's rows are spread evenly over its tiles, in steps of 32 rows (160 rows make
        // tiles of 96 and 64, not 128 and 32), so consecutive tiles cost about the same
        const int step = min(kTile, ((len + count - 1) / count + 31) & ~31);
        pv.tile_doc[base + x] = doc0 + id;
        pv.tile_row0[base + x] = row0 + t * step;
        pv.tile_len[base + x] = min(step, len - t * step);
    }

    // ---- rotation tables: cos, sin of (dst - src) * theta^(-2p/D) -------------------------------
    // thread = (slice p, every (nthreads / half)-th rank): the frequency is read once per thread
    {
        const int p = tid & (half - 1);
        const unsigned long long turns = inv_freq.turns[p];
        const double freq = inv_freq.f[p];
        for (int r = tid >> half_log2; r < n_kept; r += nthreads >> half_log2) {
            const int id = s_ids[r];
            const int delta = s_dst[id] - s_src[id];
            float2 entry;
            if (gv.dtype == CF_BF16) {
                sincos_turns(delta, turns, entry.y, entry.x);
            } else {
                double sn, cs;
                sincos_reduced((double)delta * freq, sn, cs);
                entry = make_float2((float)cs, (float)sn);
            }
            pv.trig[(size_t)(doc0 + id) * half + p] = entry;
        }
    }
}

// Clears the status words of a plan (a one-thread kernel: a kernel node after a kernel node costs
// less than a memset node between two kernels).
__global__ void clear_status_kernel(int* status) {
    status[0] = status[1] = status[2] = status[3] = 0;
}

int launch_clear_status(const PlanView& pv, cudaStream_t stream) {
    clear_status_kernel<<<1, 1, 0, stream>>>(pv.status);
    return cudaGetLastError() == cudaSuccess ? CF_OK : CF_ERR_CUDA;
}

int launch_plan(const GeomView& gv, const BatchView& bv, const PlanView& pv, int mode,
                const int* order, const int* kept_count, int query_start, const float* score_accum,
                int keep, const int* keep_per_request, int strategy, cudaStream_t stream) {
    if (gv.head_dim > 128) return CF_ERR_UNSUPPORTED;
    InvFreq inv_freq;
    for (int p = 0; p < gv.head_dim / 2; ++p) {
        inv_freq.f[p] = std::pow(gv.rope_theta, -2.0 * (double)p / (double)gv.head_dim);
        const long double turn = (long double)inv_freq.f[p] / (2.0L * 3.14159265358979323846264338327950288L);
        inv_freq.turns[p] = (unsigned long long)ldexpl(turn, 64);          // < 2^62: theta > 1 keeps f <= 1
    }
    // one thread per document of a request; barriers and scans cost less in a small block, the rotation tables (64 slices
    // per kept document) want many threads: 256 is the measured optimum for batches of up to 256 documents
    const int threads = std::min(kPlanThreads, std::max(256, (std::min(bv.n_docs_total, kMaxDocs) + 31) / 32 * 32));
    plan_kernel<<<bv.n_requests, threads, 0, stream>>>(gv, bv, pv, inv_freq, mode, order, kept_count,
                                                           query_start, score_accum, keep,
                                                           keep_per_request, strategy);
    return cudaGetLastError() == cudaSuccess ? CF_OK : CF_ERR_CUDA;
}

}  // namespace cf
