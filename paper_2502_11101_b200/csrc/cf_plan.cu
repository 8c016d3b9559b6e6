// Device-side bookkeeping of a request batch: the kept list and its order (Algorithm 2:
// Init, argsort of S, prun), the positional allocation of the kept documents (Sec. 2.3.1 Eq. 6,
// Sec. 2.5), and what the hot kernels consume: per-document rotation tables (Eq. 2 angles of
// the delta of Eq. 5) and the list of key tiles.  One thread block per request; everything
// runs in stream order so a layer stack needs no host round trip between layers.
#include <cmath>

#include "cf_common.cuh"

namespace cf {

constexpr int kPlanThreads = 256;
static_assert(4 * kPlanThreads >= kMaxDocs, "the tile scan gives four ranks to every thread");

__device__ __forceinline__ void raise_status(int* status, int code) { atomicCAS(status, 0, code); }

// Rotary frequencies theta^(-2p/D), p < D/2 (Eq. 2), computed once on the host in fp64.
struct InvFreq {
    double f[64];
};

// cos and sin of an fp64 angle to about 2e-9 absolute, for |x| up to ~1e5 (positions times a
// frequency <= 1): two-step Cody-Waite reduction by pi/2, then the Taylor polynomials of sin and
// cos on [-pi/4, pi/4] (remainders x^11/11! < 2e-9 and x^12/12! < 2e-10).  The table entries are
// rounded to fp32 afterwards, so this is as good as a correctly rounded fp64 routine at a fraction
// of its fp64 instruction count.
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

// mode 0: initialise from (order, kept_count); mode 1: prune by score, then rebuild.
// Everything a later step needs from global memory is staged in shared memory at the start, so
// the steps below do not each wait for a round trip of their own.
__global__ void __launch_bounds__(kPlanThreads)
plan_kernel(GeomView gv, BatchView bv, PlanView pv, InvFreq inv_freq, int mode, const int* __restrict__ order,
            const int* __restrict__ kept_count_in, int query_start_arg,
            const float* __restrict__ score_accum, int keep, const int* __restrict__ keep_per_request,
            int strategy) {
    __shared__ int s_ids[kMaxDocs];       // kept local ids by rank
    __shared__ int s_tmp[kMaxDocs];       // new order, then the first tile of every rank
    __shared__ int s_row[kMaxDocs + 1];   // first store row of every document (by local id), and the end
    __shared__ int s_dst[kMaxDocs];       // start positions by local id
    __shared__ int s_src[kMaxDocs];       // positions the documents were cached at, by local id
    __shared__ float s_score[kMaxDocs];
    __shared__ unsigned char s_flag[kMaxDocs];
    __shared__ int s_longest, s_min_cursor, s_fail;
    __shared__ int s_warp_sum[kPlanThreads / 32];

    const int b = blockIdx.x;
    const int tid = threadIdx.x;
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

    // ---- stage the inputs -------------------------------------------------------------------
    int n_old = 0, keep_b = 0, n_kept = 0;
    if (mode == 0) {
        n_kept = kept_count_in ? kept_count_in[b] : n_docs;
        n_kept = max(0, min(n_kept, n_docs));
        for (int r = tid; r < n_kept; r += kPlanThreads) {
            int id = order ? order[doc0 + r] : r;
            if (id < 0 || id >= n_docs) {
                raise_status(pv.status, CF_ERR_INVALID_ARG);
                id = 0;
            }
            s_ids[r] = id;
        }
    } else {
        n_old = max(0, min(pv.kept_count[b], n_docs));
        keep_b = keep_per_request ? keep_per_request[b] : keep;
        keep_b = max(0, min(keep_b, n_old));
        for (int r = tid; r < n_old; r += kPlanThreads) {
            const int id = max(0, min(pv.kept[doc0 + r], n_docs - 1));
            s_ids[r] = id;
            s_score[r] = score_accum[doc0 + id];
        }
    }
    for (int i = tid; i <= n_docs; i += kPlanThreads) s_row[i] = bv.doc_offsets[doc0 + i];
    for (int i = tid; i < n_docs; i += kPlanThreads) {
        s_src[i] = bv.doc_src_start[doc0 + i];
        s_dst[i] = mode == 0 ? -1 : pv.dst_start[doc0 + i];
    }
    int query_start = mode == 0 ? (query_start_arg < 0 ? gv.pos_range - bv.tail_reserve : query_start_arg)
                                : pv.query_start[b];
    int windows = mode == 0 ? max(1, bv.n_reuse) : pv.n_reuse[b];
    if (tid == 0) {
        s_longest = 0;
        s_min_cursor = 0x7fffffff;
        s_fail = 0;
    }
    __syncthreads();

    // ---- the kept list, in rank order -------------------------------------------------------
    if (mode != 0) {
        // rank by counting: how many kept documents beat this one (ties: lower id wins)
        for (int r = tid; r < n_old; r += kPlanThreads) {
            const float sc = s_score[r];
            const int id = s_ids[r];
            int better = 0;
            for (int o = 0; o < n_old; ++o) {
                const float so = s_score[o];
                better += (so > sc) || (so == sc && s_ids[o] < id);
            }
            s_flag[r] = better < keep_b;
            if (strategy == CF_ALLOC_SORT && better < keep_b) s_tmp[better] = id;
        }
        __syncthreads();
        if (strategy != CF_ALLOC_SORT) {
            for (int r = tid; r < n_old; r += kPlanThreads) {
                if (!s_flag[r]) continue;
                int before = 0;
                for (int o = 0; o < r; ++o) before += s_flag[o];
                s_tmp[before] = s_ids[r];
            }
        }
        __syncthreads();
        n_kept = keep_b;
        // (the clamp only matters for malformed input -- duplicate ids, NaN scores -- where two
        //  documents can claim one slot and leave another unwritten)
        for (int r = tid; r < n_kept; r += kPlanThreads) s_ids[r] = max(0, min(s_tmp[r], n_docs - 1));
        __syncthreads();
    }

    // ---- documents that are not kept ----------------------------------------------------------
    const bool reallocate = (mode == 0) || (strategy != CF_ALLOC_NONE);
    for (int i = tid; i < n_docs; i += kPlanThreads) s_flag[i] = 0;
    __syncthreads();
    for (int r = tid; r < n_kept; r += kPlanThreads) s_flag[s_ids[r]] = 1;
    __syncthreads();
    for (int i = tid; i < n_docs; i += kPlanThreads) {
        pv.doc_tile_count[doc0 + i] = 0;
        pv.doc_tile_begin[doc0 + i] = 0;
        if (!s_flag[i]) {
            pv.dst_start[doc0 + i] = -1;
            pv.group[doc0 + i] = -1;
        }
    }

    // ---- positional allocation ----------------------------------------------------------------
    if (reallocate && n_kept > 0) {
        int longest = 0;
        for (int r = tid; r < n_kept; r += kPlanThreads) longest = max(longest, s_row[s_ids[r] + 1] - s_row[s_ids[r]]);
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
        // one thread per window walks its ranks r = w, w + windows, ... backwards from the query
        for (int w = tid; w < windows && w < n_kept; w += kPlanThreads) {
            int cursor = query_start;
            for (int r = w; r < n_kept; r += windows) {
                const int id = s_ids[r];
                cursor -= s_row[id + 1] - s_row[id];
                s_dst[id] = cursor;
                pv.dst_start[doc0 + id] = cursor;
                pv.group[doc0 + id] = w;
            }
            atomicMin(&s_min_cursor, cursor);
        }
        __syncthreads();
        if (tid == 0 && (s_min_cursor < bv.prefix_len || query_start + bv.tail_reserve > gv.pos_range))
            raise_status(pv.status, CF_ERR_RANGE);
    }

    // ---- key tiles: runs of at most kTile rows that never straddle two documents -----------------
    // exclusive prefix sum of the per-rank tile counts: four consecutive ranks per thread
    int cnt[4], local = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int r = 4 * tid + k;
        cnt[k] = r < n_kept ? (s_row[s_ids[r] + 1] - s_row[s_ids[r]] + kTile - 1) / kTile : 0;
        local += cnt[k];
    }
    int incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, incl, o);
        if ((tid & 31) >= o) incl += up;
    }
    if ((tid & 31) == 31) s_warp_sum[tid >> 5] = incl;
    __syncthreads();
    int run = incl - local, total = 0;
    for (int w = 0; w < kPlanThreads / 32; ++w) {
        if (w < (tid >> 5)) run += s_warp_sum[w];
        total += s_warp_sum[w];
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int r = 4 * tid + k;
        if (r < n_kept) s_tmp[r] = run;
        run += cnt[k];
    }
    const int base = tile_base(doc0, s_row[0]);
    if (tid == 0) {
        if (base + total > pv.max_tiles) {    // cannot happen with a plan sized by cf_plan_layout_of
            raise_status(pv.status, CF_ERR_WORKSPACE);
            s_fail = 1;
        }
        const bool fail = base + total > pv.max_tiles;
        pv.n_tiles[b] = fail ? 0 : total;
        pv.kept_count[b] = fail ? 0 : n_kept;
        pv.tile_begin[b] = base;
        pv.n_reuse[b] = windows;
        pv.query_start[b] = query_start;
    }
    __syncthreads();
    if (s_fail) return;
    for (int r = tid; r < n_kept; r += kPlanThreads) {
        const int id = s_ids[r];
        const int i = doc0 + id;
        const int row0 = s_row[id];
        const int len = s_row[id + 1] - row0;
        const int first = base + s_tmp[r];
        const int count = (len + kTile - 1) / kTile;
        pv.kept[doc0 + r] = id;
        pv.doc_tile_begin[i] = first;
        pv.doc_tile_count[i] = count;
        // the document's rows are spread evenly over its tiles, in steps of 32 rows (160 rows make
        // tiles of 96 and 64, not 128 and 32), so consecutive tiles cost about the same
        const int step = count > 0 ? min(kTile, ((len + count - 1) / count + 31) & ~31) : kTile;
        for (int k = 0; k < count; ++k) {
            pv.tile_doc[first + k] = i;
            pv.tile_row0[first + k] = row0 + k * step;
            pv.tile_len[first + k] = min(step, len - k * step);
        }
    }

    // ---- rotation tables: cos, sin of (dst - src) * theta^(-2p/D), angle in fp64 --------------
    for (int idx = tid; idx < n_kept * half; idx += kPlanThreads) {
        const int r = idx / half, p = idx - r * half;
        const int id = s_ids[r];
        const double delta = (double)(s_dst[id] - s_src[id]);
        double sn, cs;
        sincos_reduced(delta * inv_freq.f[p], sn, cs);
        pv.trig[(size_t)(doc0 + id) * half + p] = make_float2((float)cs, (float)sn);
    }
}

int launch_plan(const GeomView& gv, const BatchView& bv, const PlanView& pv, int mode,
                const int* order, const int* kept_count, int query_start, const float* score_accum,
                int keep, const int* keep_per_request, int strategy, cudaStream_t stream) {
    if (gv.head_dim > 128) return CF_ERR_UNSUPPORTED;
    InvFreq inv_freq;
    for (int p = 0; p < gv.head_dim / 2; ++p)
        inv_freq.f[p] = std::pow(gv.rope_theta, -2.0 * (double)p / (double)gv.head_dim);
    plan_kernel<<<bv.n_requests, kPlanThreads, 0, stream>>>(gv, bv, pv, inv_freq, mode, order, kept_count,
                                                           query_start, score_accum, keep,
                                                           keep_per_request, strategy);
    return cudaGetLastError() == cudaSuccess ? CF_OK : CF_ERR_CUDA;
}

}  // namespace cf
