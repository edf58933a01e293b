// s4c_tree_accept_filtered: speculative-sampling acceptance (Section 2; Eq. 11, Eq. 12; longest accepted path,
// Section 3.2) against a top-k / nucleus FILTERED target distribution -- the sampling regime of Section 4 (RQ5).
//
// Filtering makes the target distribution sparse: at most top_k (<= 64) tokens per node keep any mass.  So the only
// vocabulary-wide work is finding those tokens -- a selection over the logits that needs no exponential -- and the mass
// of every draft row (the renormalisation after a rejection needs it).  Three kernels, the second and third launched
// programmatically dependent on their predecessor:
//   filter_span_kernel   One streaming pass over logits and draft probabilities (HBM-bound by design: 8 bytes per
//                        vocabulary entry).  All rows' batches of 4096 entries form one list that is cut into equal
//                        runs, one CTA per run and as many CTAs as the GPU holds at once; a run that crosses into the
//                        next row ends a piece of the one and starts a piece of the other.  Per piece a CTA keeps a POOL
//                        of the entries at or above a THRESHOLD that only rises: for the first batch the threshold is
//                        the smallest of the maxima of 256/G groups of G threads (at least k entries lie at or above
//                        it); the pool is then cut back to its k best -- a 256-bin histogram over [threshold, maximum],
//                        the bin where the count from the top reaches k, exact ranks (logit descending, token ascending)
//                        by counting among the few entries of the bins down to it -- and the threshold becomes the k-th
//                        best.  Later batches only compare with the threshold (whole warps usually find nothing), push
//                        what passes, and the pool is cut back again when it has grown.  Between the sync points (every
//                        fourth batch) warps run apart, each with its next batch's loads in flight.  Pieces that this
//                        cannot serve (heavy ties, masked vocabularies: more than the pool or the ranking holds) are
//                        redone on an exact path: every thread sorts its 16 entries of a batch, warps merge their lanes'
//                        lists head by head, one warp merges the warps' lists with the best so far.  Output per piece:
//                        its k best, sorted, and its draft mass in float64.
//   filter_rows_kernel   grid (T, B): merges a row's pieces pairwise (a bitonic merge of two sorted lists in a warp's
//                        registers, a tree of such merges) into the row's k best, turns them into probabilities in
//                        float64 (softmax over the kept logits at the temperature), cuts the nucleus and renormalises:
//                        per node a short list (token, probability, draft probability) in rank order, and the draft
//                        row's mass
//   accept_walk_sparse_kernel  grid (B): the walk of s4c_tree_accept on these lists, by one warp: acceptance tests,
//                        residual masses and the final inverse-CDF draw run over the <= 64 kept tokens of a node.
// HBM traffic: every logits row and every draft row once.  Ranking, sums and decisions are deterministic (fixed orders);
// ties between equal logits go to the lower token.  No tensor cores: there is no contraction here.
#include <float.h>
#include <limits.h>
#include <math.h>

#include <algorithm>

#include "s4c_common.cuh"

namespace s4c {

constexpr int kFsThreads = 256;
constexpr int kFsElems = 16;
constexpr int kFsSeg = kFsThreads * kFsElems;  // 4096 logits per CTA
constexpr int kMaxTopK = 64;

struct __align__(8) FCand {  // a candidate: logit and token; (-inf, INT_MAX) = none
    float x;
    int tok;
};
__device__ __forceinline__ bool f_before(float a, int at, float b, int bt) { return a > b || (a == b && at < bt); }

// One warp merges up to 32 sorted lists (lane l owns list l: entry h at lists[h * h_stride + l * l_stride], `len`
// entries each, best first; n_lists >= 1, len >= 1) into the k best overall, written to out[0..k) (best first;
// (-inf, INT_MAX) when the lists run out).  Tokens are distinct across lists.  Every lane reloads its current entry
// every round, from an index that is always inside a list (lanes without a list read list 0 and discard what they read).
__device__ __forceinline__ void merge_heads(const FCand* lists, int n_lists, int len, int h_stride, int l_stride, int k,
                                            FCand* out) {
    const int lane = threadIdx.x & 31;
    const bool mine = lane < n_lists;
    const FCand* my = lists + (mine ? lane : 0) * l_stride;  // this lane's list: entry h at my[h * h_stride]
    int head = 0;
    FCand c = my[0];
    float cx = mine ? c.x : -INFINITY;
    int ct = mine ? c.tok : INT_MAX;
    for (int r = 0; r < k; ++r) {
        float bx = cx;
        int bt = ct;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ox = __shfl_xor_sync(0xffffffffu, bx, o);
            const int ot = __shfl_xor_sync(0xffffffffu, bt, o);
            if (f_before(ox, ot, bx, bt)) bx = ox, bt = ot;
        }
        if (lane == 0) {
            out[r].x = bt == INT_MAX ? -INFINITY : bx;
            out[r].tok = bt;
        }
        head += (bt != INT_MAX && ct == bt) ? 1 : 0;  // the winner moves on to its next entry
        const bool more = mine && head < len;
        c = my[(more ? head : 0) * h_stride];
        cx = more ? c.x : -INFINITY;
        ct = more ? c.tok : INT_MAX;
    }
}

// programmatic dependent launch: the three kernels of a call overlap their launch latencies and prologues
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float fmax_keep_nan(float a, float b) {
    float d;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}

// order-preserving map of a float onto unsigned integers (a > b  <=>  key(a) > key(b); -0 ranks just below +0, which
// only shifts a threshold by nothing that can be told apart: thresholds are compared as floats again)
__device__ __forceinline__ uint32_t f_key(float x) {
    const uint32_t u = __float_as_uint(x);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float f_unkey(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
constexpr uint32_t kKeyNegInf = 0x007fffffu;  // f_key(-inf)

constexpr int kFsBins = 256;   // histogram bins of the threshold selection
constexpr int kFsCap = 256;    // most candidates ranked by counting
constexpr int kFsList = 1024;  // most entries at or above the threshold that the selection handles

constexpr int kFsSelect = 384;  // the pool is cut back to its k best when it has grown beyond this
constexpr int kFsSyncEvery = 4; // batches between two looks at the pool

struct __align__(16) SpanShared {
    union {
        FCand lists[kFsElems][kFsThreads];  // exact path: entry h of thread t at [h][t]
        struct {
            int hist[kFsBins];
            FCand cand[kFsCap];
            FCand pool[kFsList];    // entries at or above the threshold: the k best so far and what came in since
            uint8_t qbin[kFsList];  // their bins
        } fast;
    };
    FCand wlist[kFsThreads / 32 + 1][kMaxTopK];  // exact path: the warps' k best of a batch; last row: the k best so far
    FCand sorted[kMaxTopK];                       // the result of a selection, best first
    uint32_t wmax[kFsThreads / 32], wmin[kFsThreads / 32];
    int wfin[kFsThreads / 32];
    double wq[kFsThreads / 32];
    int ncand, npool, snap, bad;
    uint32_t poolmax;
};

// The k best of the pool (all entries >= lo), best first, into sh.sorted; every thread of the CTA calls it after a
// barrier that completed the pool.  Returns how many there are (min(k, n_pool)), or -1 if more than kFsCap entries share
// the bins down to the k-th (heavy ties: the caller takes the exact path).
__device__ __forceinline__ int select_from_pool(SpanShared& sh, int n_pool, float lo, int k) {
    const int tid = threadIdx.x, lane = tid & 31;
    const FCand* src = sh.fast.pool;
    int n_cand = n_pool;
    if (n_pool > kFsCap) {
        sh.fast.hist[tid] = 0;  // kFsBins == kFsThreads
        if (tid == 0) sh.poolmax = 0, sh.ncand = 0;
        __syncthreads();
        uint32_t km = 0;
        for (int t = tid; t < n_pool; t += kFsThreads) km = max(km, f_key(sh.fast.pool[t].x));
        km = __reduce_max_sync(0xffffffffu, km);
        if (lane == 0) atomicMax(&sh.poolmax, km);
        __syncthreads();
        // 256 bins over [lo, M]; bins fall with the logit (float subtraction, multiplication by a positive constant and
        // truncation are monotone) and equal logits share a bin
        const float M = f_unkey(sh.poolmax);
        const float inv = (float)kFsBins / (M - lo);
        for (int t = tid; t < n_pool; t += kFsThreads) {
            const int bin = max(0, min(kFsBins - 1, (int)((M - sh.fast.pool[t].x) * inv)));  // (int)NaN = 0: M == lo
            sh.fast.qbin[t] = (uint8_t)bin;
            atomicAdd(&sh.fast.hist[bin], 1);
        }
        __syncthreads();
        // every warp finds the bin where the count from the top reaches k (the same scan in every warp: no broadcast)
        const int4 h0 = *reinterpret_cast<const int4*>(&sh.fast.hist[lane * 8]);
        const int4 h1 = *reinterpret_cast<const int4*>(&sh.fast.hist[lane * 8 + 4]);
        const int c8[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
        const int mine = (h0.x + h0.y) + (h0.z + h0.w) + (h1.x + h1.y) + (h1.z + h1.w);
        int cum = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, cum, o);
            if (lane >= o) cum += up;
        }
        const uint32_t reach = __ballot_sync(0xffffffffu, cum >= k);  // not empty: the bins hold n_pool > k entries
        const int L = __ffs(reach) - 1;
        int bstar = 0, ctot = 0;
        if (lane == L) {
            int run = cum - mine;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                run += c8[j];
                if (run >= k && ctot == 0) bstar = lane * 8 + j, ctot = run;
            }
        }
        bstar = __shfl_sync(0xffffffffu, bstar, L), ctot = __shfl_sync(0xffffffffu, ctot, L);
        if (ctot > kFsCap) return -1;
        for (int t = tid; t < n_pool; t += kFsThreads)
            if (sh.fast.qbin[t] <= bstar) sh.fast.cand[atomicAdd(&sh.ncand, 1)] = sh.fast.pool[t];
        __syncthreads();
        src = sh.fast.cand, n_cand = ctot;
    }
    // exact ranks among the candidates by counting (the order is total: the ranks are 0 .. n_cand-1); up to four threads
    // share a candidate
    const int parts = n_cand <= 64 ? 4 : (n_cand <= 128 ? 2 : 1);
    const int idx = tid / parts, sub = tid % parts;
    const FCand me = src[max(0, min(idx, n_cand - 1))];
    int r = 0;
#pragma unroll 4
    for (int j = sub; j < n_cand; j += parts) {
        const FCand o = src[j];
        r += f_before(o.x, o.tok, me.x, me.tok) ? 1 : 0;
    }
    if (parts > 1) r += __shfl_xor_sync(0xffffffffu, r, 1);
    if (parts > 2) r += __shfl_xor_sync(0xffffffffu, r, 2);
    if (sub == 0 && idx < n_cand && r < k) sh.sorted[r] = me;
    __syncthreads();
    return min(k, n_cand);
}

// The exact path for a piece (batches batch0 .. batch1-1 of one row) that the streaming selection cannot serve: every
// thread sorts its 16 entries of a batch, warps merge their lanes' lists head by head, one warp merges the warps' lists
// with the k best so far.  Its own function, not inlined: it needs twice the registers of the streaming loop and runs
// only for tie-heavy or masked pieces.  Leaves the piece's k best in sh.sorted; returns the thread's share of the draft
// mass in *qs and whether the piece holds a NaN or +Inf.
template <bool VEC>
__device__ __noinline__ bool exact_piece(SpanShared& sh, const float* __restrict__ row, const float* __restrict__ qrow, int V,
                                         int k, int batch0, int batch1, double* qs_out) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    double qs = 0.0;
    bool unusable = false;
    FCand* best = sh.wlist[kFsThreads / 32];
    for (int r = tid; r < kMaxTopK; r += kFsThreads) best[r].x = -INFINITY, best[r].tok = INT_MAX;
    for (int batch = batch0; batch < batch1 && !unusable; ++batch) {
        const int s0 = batch * kFsSeg;
        float x[kFsElems];
        int e[kFsElems];
        bool bad_here = false;
#pragma unroll
        for (int i = 0; i < kFsElems; ++i) {
            const int tok = VEC ? s0 + ((i >> 2) * kFsThreads + tid) * 4 + (i & 3) : s0 + i * kFsThreads + tid;
            const bool in = tok < V;
            x[i] = in ? __ldg(row + tok) : -INFINITY;
            qs += in ? (double)__ldg(qrow + tok) : 0.0;
            e[i] = in ? tok : INT_MAX;  // slots past the row rank last
            bad_here = bad_here || !(x[i] < INFINITY);
        }
        // sort the thread's 16 entries, best first (bitonic network on (logit, token) pairs; the order is total)
#pragma unroll
        for (int size = 2; size <= kFsElems; size <<= 1)
#pragma unroll
            for (int stride = size >> 1; stride > 0; stride >>= 1)
#pragma unroll
                for (int i = 0; i < kFsElems; ++i) {
                    const int j = i ^ stride;
                    if (j > i) {
                        const bool up = (i & size) == 0;  // this block sorts best-first, its sibling worst-first
                        const bool swap = up ? f_before(x[j], e[j], x[i], e[i]) : f_before(x[i], e[i], x[j], e[j]);
                        if (swap) {
                            const float tx = x[i];
                            x[i] = x[j], x[j] = tx;
                            const int te = e[i];
                            e[i] = e[j], e[j] = te;
                        }
                    }
                }
#pragma unroll
        for (int i = 0; i < kFsElems; ++i) sh.lists[i][tid].x = x[i], sh.lists[i][tid].tok = e[i];
        __syncwarp();
        merge_heads(&sh.lists[0][warp * 32], 32, kFsElems, kFsThreads, 1, k, sh.wlist[warp]);
        unusable = __syncthreads_or(bad_here);
        if (warp == 0) {  // nine lists: the warps' and the best so far; the result replaces the best so far
            merge_heads(&sh.wlist[0][0], kFsThreads / 32 + 1, k, 1, kMaxTopK, k, sh.sorted);
            __syncwarp();
            for (int r = lane; r < k; r += 32) best[r] = sh.sorted[r];
        }
        __syncthreads();
    }
    *qs_out = qs;
    return unusable;
}

// The rows' batches (4096 entries each) form one long list, cut into equal runs of `per` batches: one CTA per run, all
// CTAs resident at once, every CTA with the same amount to read.  A run that crosses from one row into the next ends a
// piece and starts another; a row is covered by at most pmax pieces.  For every piece: the k best logits (sorted) and the
// draft mass.
template <bool VEC>
__global__ void __launch_bounds__(kFsThreads, 3)
filter_span_kernel(const float* __restrict__ logits, const float* __restrict__ dprobs, const int32_t* __restrict__ n_nodes,
                   int n_rows, int T, int V, int k, int G, int per, int pmax, FCand* __restrict__ cand,
                   double* __restrict__ qpart) {
    griddep_launch_dependents();  // the next kernel of the call may become resident; it waits for this grid's completion
    __shared__ SpanShared sh;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_batches = (V + kFsSeg - 1) / kFsSeg;
    const long long run0 = (long long)blockIdx.x * per, run1 = min((long long)n_rows * n_batches, run0 + per);
    const float* row = nullptr;
    const float* qrow = nullptr;
    // entry i of this thread in the batch that starts at token s0 is token tok_of(s0, i); the same map on every path
    auto tok_of = [&](int s0, int i) {
        return VEC ? s0 + ((i >> 2) * kFsThreads + tid) * 4 + (i & 3) : s0 + i * kFsThreads + tid;
    };
    float x[kFsElems];
    double qs = 0.0;
    auto load_batch = [&](int s0) {  // logits into x[], the draft probabilities into the running sum
        if (VEC) {  // V % 4 == 0: whole 16-byte words, all requested before any is used
            float4 lv[kFsElems / 4], qv[kFsElems / 4];
#pragma unroll
            for (int i = 0; i < kFsElems / 4; ++i) {
                lv[i] = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY), qv[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (tok_of(s0, 4 * i) < V) {
                    lv[i] = __ldg(reinterpret_cast<const float4*>(row + tok_of(s0, 4 * i)));
                    qv[i] = __ldg(reinterpret_cast<const float4*>(qrow + tok_of(s0, 4 * i)));
                }
            }
#pragma unroll
            for (int i = 0; i < kFsElems / 4; ++i) {
                x[4 * i + 0] = lv[i].x, x[4 * i + 1] = lv[i].y, x[4 * i + 2] = lv[i].z, x[4 * i + 3] = lv[i].w;
                qs += ((double)qv[i].x + (double)qv[i].y) + ((double)qv[i].z + (double)qv[i].w);
            }
        } else {
            float q[kFsElems];
#pragma unroll
            for (int i = 0; i < kFsElems; ++i) {
                const bool in = tok_of(s0, i) < V;
                x[i] = in ? __ldg(row + tok_of(s0, i)) : -INFINITY;
                q[i] = in ? __ldg(qrow + tok_of(s0, i)) : 0.f;
            }
#pragma unroll
            for (int i = 0; i < kFsElems; ++i) qs += (double)q[i];
        }
    };

    for (long long run = run0; run < run1;) {
        // ---- one piece: batches batch0 .. batch1-1 of row `at`
        const size_t at = (size_t)(run / n_batches);  // the row: sequence * T + node
        const int batch0 = (int)(run - (long long)at * n_batches);
        const int batch1 = (int)min((long long)n_batches, batch0 + (run1 - run));
        run += batch1 - batch0;
        if (n_nodes && (int)(at % T) >= n_nodes[at / T]) continue;
        row = logits + at * V, qrow = dprobs + at * V;
        const int piece = blockIdx.x - (int)(((long long)at * n_batches) / per);  // CTAs before this one on the same row
        FCand* out = cand + (at * pmax + piece) * k;
        qs = 0.0;
        // ---- the streaming path: a pool of entries at or above a threshold that only rises
        if (tid == 0) sh.npool = 0, sh.bad = 0;
        __syncthreads();
        bool exact_path = false, unusable = false, selected_last = false;
        int kk = 0;              // entries in sh.sorted after the last selection
        float lo = -INFINITY;    // the threshold: nothing below it is among the k best of what was seen so far
        bool have_lo = false;
        // (16-byte words: the next batch's loads are issued before this batch is worked on, so that a warp always has loads
        // in flight)
        float4 lv[kFsElems / 4], qv[kFsElems / 4];
        auto issue = [&](int s0) {
            const float4* la = reinterpret_cast<const float4*>(row + s0) + tid;  // word i of this thread: la[i * 256]
            const float4* qa = reinterpret_cast<const float4*>(qrow + s0) + tid;
            if (s0 + kFsSeg <= V) {  // a whole batch: no bounds to check, constant offsets
#pragma unroll
                for (int i = 0; i < kFsElems / 4; ++i) lv[i] = __ldg(la + i * kFsThreads), qv[i] = __ldg(qa + i * kFsThreads);
            } else {
#pragma unroll
                for (int i = 0; i < kFsElems / 4; ++i) {
                    lv[i] = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY), qv[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (tok_of(s0, 4 * i) < V) lv[i] = __ldg(la + i * kFsThreads), qv[i] = __ldg(qa + i * kFsThreads);
                }
            }
        };
        if (VEC) issue(batch0 * kFsSeg);
        for (int batch = batch0; batch < batch1; ++batch) {
            const int s0 = batch * kFsSeg;
            if (VEC) {
#pragma unroll
                for (int i = 0; i < kFsElems / 4; ++i) {
                    x[4 * i + 0] = lv[i].x, x[4 * i + 1] = lv[i].y, x[4 * i + 2] = lv[i].z, x[4 * i + 3] = lv[i].w;
                    qs += ((double)qv[i].x + (double)qv[i].y) + ((double)qv[i].z + (double)qv[i].w);
                }
                if (batch + 1 < batch1) issue(s0 + kFsSeg);
            } else {
                load_batch(s0);
            }
            float mx = x[0];
#pragma unroll
            for (int i = 1; i < kFsElems; ++i) mx = fmax_keep_nan(mx, x[i]);  // a NaN survives
            const bool bad_here = !(mx < INFINITY);  // NaN or +Inf: the row is unusable
            if (bad_here) sh.bad = 1;
            if (!have_lo) {
                // The first threshold.  Threads form groups of G (the largest power of two that leaves 256 / G >= k groups);
                // every group holds an entry equal to its maximum, so at least as many entries as there are groups with a
                // finite maximum lie at or above the smallest such maximum: with k or more of those groups nothing below it
                // is among the k best.
                const uint32_t key = bad_here ? 0xffffffffu : f_key(mx);
                const int Gw = min(G, 32);
                uint32_t gk = key;
                for (int o = 1; o < Gw; o <<= 1) gk = max(gk, __shfl_xor_sync(0xffffffffu, gk, o));
                const bool fin = gk > kKeyNegInf;  // the group (its part in this warp) holds something above -inf
                const uint32_t kmax = __reduce_max_sync(0xffffffffu, key);
                const uint32_t kmin = __reduce_min_sync(0xffffffffu, fin ? gk : 0xffffffffu);
                const int nfin_w = __popc(__ballot_sync(0xffffffffu, fin && (lane & (Gw - 1)) == 0));
                if (lane == 0) sh.wmax[warp] = kmax, sh.wmin[warp] = kmin, sh.wfin[warp] = nfin_w;
                __syncthreads();
                uint32_t Kmin = 0xffffffffu;
                int n_fin = 0;
                if (G <= 32) {
#pragma unroll
                    for (int w = 0; w < kFsThreads / 32; ++w) Kmin = min(Kmin, sh.wmin[w]), n_fin += sh.wfin[w];
                } else {  // a group is G / 32 whole warps
                    const int W = G >> 5;
                    for (int g = 0; g < kFsThreads / 32; g += W) {
                        uint32_t gm = 0;
                        for (int w = g; w < g + W; ++w) gm = max(gm, sh.wmax[w]);
                        if (gm > kKeyNegInf) Kmin = min(Kmin, gm), ++n_fin;
                    }
                }
                if (n_fin >= k) lo = f_unkey(Kmin);  // else everything in the batch is a candidate (lo stays -inf)
                have_lo = true;
            }
            // entries at or above the threshold go to the pool: count, one slot range per warp, write.  No CTA barrier here:
            // between the sync points below the warps run apart, each with its next batch's loads in flight.
            // (a thread whose maximum is below the threshold has nothing to give: in the steady state whole warps skip this)
            if (__any_sync(0xffffffffu, mx >= lo)) {
                const bool ragged = s0 + kFsSeg > V;  // the row ends inside this batch: slots past it are not entries
                int c = 0;
                if (!ragged) {
#pragma unroll
                    for (int i = 0; i < kFsElems; ++i) c += x[i] >= lo ? 1 : 0;
                } else {
#pragma unroll
                    for (int i = 0; i < kFsElems; ++i) c += (x[i] >= lo && tok_of(s0, i) < V) ? 1 : 0;
                }
                if (__any_sync(0xffffffffu, c > 0)) {
                    int incl = c;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const int up = __shfl_up_sync(0xffffffffu, incl, o);
                        if (lane >= o) incl += up;
                    }
                    int wbase = 0;
                    if (lane == 31) wbase = atomicAdd(&sh.npool, incl);
                    wbase = __shfl_sync(0xffffffffu, wbase, 31);
                    int off = wbase + incl - c;
                    if (c > 0) {
#pragma unroll
                        for (int i = 0; i < kFsElems; ++i)
                            if (x[i] >= lo && (!ragged || tok_of(s0, i) < V) && off < kFsList) {
                                sh.fast.pool[off].x = x[i], sh.fast.pool[off].tok = tok_of(s0, i);
                                ++off;
                            }
                    }
                }
            }
            // sync points: the first batch, every kFsSyncEvery-th after it and the last.  Between two of them the pool takes
            // what comes in under the threshold of the last selection (more than the best threshold would let in, never
            // less); if that overflows the pool, the span is redone on the exact path.
            if (batch != batch0 && batch != batch1 - 1 && (batch - batch0) % kFsSyncEvery != 0) continue;
            __syncthreads();  // the pool holds everything pushed so far
            if (tid == 0) sh.snap = sh.bad ? -1 : sh.npool;
            __syncthreads();  // one value for every thread, read before anybody pushes (or flags a bad entry) again
            if (sh.snap < 0) {
                unusable = true;
                break;
            }
            const int n_pool = sh.snap;
            if (n_pool > kFsList) {  // more than the pool holds (ties, a masked vocabulary)
                exact_path = true;
                break;
            }
            if (n_pool > kFsSelect || batch == batch0) {
                // cut the pool back to its k best and raise the threshold to the k-th of them
                kk = select_from_pool(sh, n_pool, lo, k);
                if (kk < 0) {
                    exact_path = true;
                    break;
                }
                if (batch == batch1 - 1) {  // the piece's result is in sh.sorted
                    selected_last = true;
                    break;
                }
                if (tid == 0) sh.npool = kk;
                if (tid < kk) sh.fast.pool[tid] = sh.sorted[tid];
                if (kk == k) lo = sh.sorted[k - 1].x;
                __syncthreads();
            }
        }
        if (!exact_path && !unusable && !selected_last) {
            // one more selection unless nothing came in since the last one (the pool is then sh.sorted already)
            const int n_pool = sh.npool;
            if (n_pool != kk || kk == 0) {
                kk = select_from_pool(sh, n_pool, lo, k);
                if (kk < 0) exact_path = true;
            }
        }
        if (exact_path) {
            __syncthreads();  // nobody reads the pool any more: its memory is reused
            unusable = exact_piece<VEC>(sh, row, qrow, V, k, batch0, batch1, &qs);  // from the start of the piece
            kk = k;  // (empty entries at the end when the piece holds fewer than k)
        }
        // ---- results: the piece's draft mass and its k best (or the mark of an unusable row)
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) qs += __shfl_xor_sync(0xffffffffu, qs, o);
        if (lane == 0) sh.wq[warp] = qs;
        __syncthreads();
        if (tid == 0) {
            double tot = 0.0;
            for (int w = 0; w < kFsThreads / 32; ++w) tot += sh.wq[w];
            qpart[at * pmax + piece] = tot;
        }
        for (int r = tid; r < k; r += kFsThreads) {
            FCand v;
            v.x = -INFINITY, v.tok = INT_MAX;
            if (unusable)  // a NaN or +Inf in the piece: +Inf in the first slot tells the row kernel (the walk flags the sequence)
                v.x = r == 0 ? INFINITY : -INFINITY, v.tok = r == 0 ? 0 : INT_MAX;
            else if (r < kk)
                v = sh.sorted[r];
            out[r] = v;
        }
        __syncthreads();  // the next piece reuses the shared state
    }
}

struct KeptLists {  // per (sequence, node): the filtered target distribution
    int32_t* n;     // [B*T]: kept tokens (1..top_k); -1: the row is unusable (NaN / +Inf logit, or nothing but -Inf)
    int32_t* tok;   // [B*T*k] in rank order
    double* p;      // [B*T*k] target probabilities
    float* q0;      // [B*T*k] the draft row's probabilities of the same tokens, as given
    double* qtot;   // [B*T] the draft row's mass
};

constexpr int kFrThreads = 512;  // 16 warps: one pair of lists each
constexpr int kFrLists = 32;     // lists merged per round

// One warp merges two sorted lists of 64 (best first; lane l holds entries l and l + 32 of the result) and keeps the
// 64 best: entry i of the one against entry 63 - i of the other leaves the 64 best as a bitonic sequence, which five
// shuffle stages and one in-lane stage sort.
__device__ __forceinline__ void merge_pair(const FCand* a, const FCand* b, FCand& c0, FCand& c1) {
    const int lane = threadIdx.x & 31;
    const FCand a0 = a[lane], a1 = a[lane + 32], b0 = b[63 - lane], b1 = b[31 - lane];
    c0 = f_before(b0.x, b0.tok, a0.x, a0.tok) ? b0 : a0;
    c1 = f_before(b1.x, b1.tok, a1.x, a1.tok) ? b1 : a1;
    if (f_before(c1.x, c1.tok, c0.x, c0.tok)) {
        const FCand t = c0;
        c0 = c1, c1 = t;
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) {
        const bool low = (lane & s) == 0;  // the lower lane of a pair keeps the better entry
        FCand o;
        o.x = __shfl_xor_sync(0xffffffffu, c0.x, s), o.tok = __shfl_xor_sync(0xffffffffu, c0.tok, s);
        if (f_before(o.x, o.tok, c0.x, c0.tok) == low) c0 = o;
        o.x = __shfl_xor_sync(0xffffffffu, c1.x, s), o.tok = __shfl_xor_sync(0xffffffffu, c1.tok, s);
        if (f_before(o.x, o.tok, c1.x, c1.tok) == low) c1 = o;
    }
}

__global__ void __launch_bounds__(kFrThreads)
filter_rows_kernel(const FCand* __restrict__ cand, const double* __restrict__ qpart, const float* __restrict__ dprobs,
                   const int32_t* __restrict__ n_nodes, int T, int V, int per, int pmax, int k, double inv_tau, double top_p,
                   KeptLists kept) {
    const int node = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    griddep_launch_dependents();
    griddep_wait();  // the segments' lists and masses are complete
    if (n_nodes && node >= n_nodes[b]) return;
    __shared__ FCand A[kFrLists][kMaxTopK];
    const size_t at = (size_t)b * T + node;
    // the row's pieces: the CTAs of the selection kernel whose runs of `per` batches meet this row's batches
    const int n_batches = (V + kFsSeg - 1) / kFsSeg;
    const int segs = (int)((((long long)at + 1) * n_batches - 1) / per - ((long long)at * n_batches) / per) + 1;
    const FCand* c = cand + at * pmax * k;
    qpart += at * pmax;
    // the row's best out of the pieces' lists: 32 lists at a time (later rounds: the best so far and 31 new ones),
    // halved by pairwise merges until one is left in A[0]
    for (int s = 0, first = 1; s < segs; first = 0) {
        const int base = first ? 0 : 1, cnt = min(kFrLists - base, segs - s);
        for (int i = tid; i < cnt * kMaxTopK; i += kFrThreads) {
            const int l = i >> 6, j = i & 63;
            FCand v;
            v.x = -INFINITY, v.tok = INT_MAX;
            if (j < k) v = c[(size_t)(s + l) * k + j];
            A[base + l][j] = v;
        }
        __syncthreads();
        for (int n = base + cnt; n > 1;) {
            const int half = (n + 1) >> 1;
            FCand c0, c1;
            if (warp < (n >> 1))
                merge_pair(A[2 * warp], A[2 * warp + 1], c0, c1);
            else if (warp < half)  // n is odd: the last list moves down as it is
                c0 = A[n - 1][lane], c1 = A[n - 1][lane + 32];
            __syncthreads();
            if (warp < half) A[warp][lane] = c0, A[warp][lane + 32] = c1;
            __syncthreads();
            n = half;
        }
        s += cnt;
    }
    if (warp == kFrThreads / 32 - 1) {  // the draft row's mass: the segments' sums in segment order (beside warp 0's work)
        double qt = 0.0;
        for (int s0 = 0; s0 < segs; s0 += 32) {
            const double v = s0 + lane < segs ? qpart[s0 + lane] : 0.0;
            const int cnt = min(32, segs - s0);
            for (int i = 0; i < cnt; ++i) qt += __shfl_sync(0xffffffffu, v, i);
        }
        if (lane == 0) kept.qtot[at] = qt;
    }
    if (warp != 0) return;
    const FCand* top = A[0];
    const float M = top[0].x;
    if (!(M > -INFINITY && M < INFINITY)) {
        if (lane == 0) kept.n[at] = -1;
        return;
    }
    // probabilities over the kept logits, sums in rank order (lane 0: at most 64 terms)
    __shared__ double ej[kMaxTopK];
    for (int j = lane; j < k; j += 32) ej[j] = top[j].tok == INT_MAX ? 0.0 : exp(((double)top[j].x - (double)M) * inv_tau);
    __syncwarp();
    __shared__ double pj[kMaxTopK];
    __shared__ int m_s;
    __shared__ double mass_s;
    // (fewer than k tokens in the vocabulary: the lists end in empty entries)
    const uint32_t real0 = __ballot_sync(0xffffffffu, lane < k && top[lane].tok != INT_MAX);
    const uint32_t real1 = __ballot_sync(0xffffffffu, lane + 32 < k && top[min(lane + 32, kMaxTopK - 1)].tok != INT_MAX);
    const int kk = __popc(real0) + __popc(real1);
    double mass = 0.0;  // every lane sums the same terms in the same (rank) order
    for (int j = 0; j < kk; ++j) mass += ej[j];
    int m = kk;
    if (top_p < 1.0) {
        for (int j = lane; j < kk; j += 32) pj[j] = ej[j] / mass;  // the divisions side by side, the sum in order
        __syncwarp();
        double cum = 0.0;
        for (int j = 0; j < kk; ++j) {
            cum += pj[j];
            if (cum >= top_p) {
                m = j + 1;
                break;
            }
        }
        mass = 0.0;
        for (int j = 0; j < m; ++j) mass += ej[j];
    }
    if (lane == 0) m_s = m, mass_s = mass, kept.n[at] = m;
    __syncwarp();
    for (int j = lane; j < k; j += 32) {
        const bool in = j < m_s;
        kept.tok[at * k + j] = in ? top[j].tok : -1;
        kept.p[at * k + j] = in ? ej[j] / mass_s : 0.0;
        kept.q0[at * k + j] = in ? __ldg(dprobs + at * V + top[j].tok) : 0.f;
    }
}

struct SparseShared {
    int32_t par[S4C_MAX_T];
    int32_t tok[S4C_MAX_T];
    float uni[S4C_MAX_T];
    int depth[S4C_MAX_T];
    uint32_t anc[S4C_MAX_T][S4C_MASK_WORDS];
    double tq0[S4C_MAX_T];   // draft probability of node i's token under its parent's row
    int ktok[kMaxTopK];      // the current node's kept tokens, in rank order
    double kp[kMaxTopK];     // their current target probabilities
    double kq0[kMaxTopK];    // their draft probabilities as given
    int kgone[kMaxTopK];     // 1: the token was rejected here and has left the draft distribution
    int order[kMaxTopK];     // the kept tokens' list positions in token order (the order the vocabulary is scanned in)
    int flag;
};

__global__ void __launch_bounds__(kFsThreads)
accept_walk_sparse_kernel(const float* __restrict__ dprobs, const int32_t* __restrict__ tokens, const int32_t* __restrict__ parent,
                          const int32_t* __restrict__ n_nodes, const float* __restrict__ uniforms, int T, int V, int k,
                          int max_depth, KeptLists kept, int32_t* __restrict__ accept_len, int32_t* __restrict__ path,
                          int32_t* __restrict__ next_token, uint8_t* __restrict__ near_tie, int32_t* __restrict__ status) {
    __shared__ SparseShared sh;
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
    const int n = n_nodes ? n_nodes[b] : T;
    int32_t* pth = path + (size_t)b * (max_depth + 1);
    for (int i = tid; i < T; i += blockDim.x) {
        sh.par[i] = parent[(size_t)b * T + i];
        sh.tok[i] = tokens[(size_t)b * T + i];
        sh.uni[i] = uniforms[(size_t)b * T + i];
        if (near_tie) near_tie[(size_t)b * T + i] = 0;
    }
    __syncthreads();
    int flags = build_ancestor_masks(sh.par, n, T, sh.anc, sh.depth, &sh.flag);
    if (!flags) {
        for (int i = tid; i < n; i += blockDim.x) {
            if (sh.tok[i] < 0 || sh.tok[i] >= V) atomicOr(&sh.flag, S4C_SEQ_TOKEN_RANGE);
            if (sh.depth[i] > max_depth) atomicOr(&sh.flag, S4C_SEQ_DEPTH);
        }
        __syncthreads();
        flags = sh.flag;
    }
    if (!flags)  // (tokens are in range) -- these reads of the caller's inputs need not wait for the lists either
        for (int i = 1 + tid; i < n; i += blockDim.x)
            sh.tq0[i] = (double)__ldg(dprobs + ((size_t)b * T + sh.par[i]) * V + sh.tok[i]);
    griddep_wait();  // the kept lists are complete
    if (!flags) {
        for (int i = tid; i < n; i += blockDim.x)
            if (kept.n[(size_t)b * T + i] < 0) atomicOr(&sh.flag, S4C_SEQ_NONFINITE);
        __syncthreads();
        flags = sh.flag;
    }
    if (tid == 0 && status) status[b] = flags;
    if (flags) {
        for (int j = tid; j <= max_depth; j += blockDim.x) pth[j] = -1;
        if (tid == 0) accept_len[b] = -1, next_token[b] = -1;
        return;
    }
    if (tid >= 32) return;  // the walk itself is one warp's work: lists of at most 64 entries, two per lane

    int cur = 0;
    for (int guard = 0; guard <= T; ++guard) {
        const size_t at = (size_t)b * T + cur;
        const int m = kept.n[at];
        double qtot = kept.qtot[at];  // mass of the draft distribution as it stands
        double qscale = 1.0;          // the draft distribution is the given row times this, rejected tokens left out
        for (int j = lane; j < k; j += 32)  // all k slots (those past m hold token -1 and no mass): no wait for m
            sh.ktok[j] = kept.tok[at * k + j], sh.kp[j] = kept.p[at * k + j], sh.kq0[j] = (double)kept.q0[at * k + j], sh.kgone[j] = 0;
        __syncwarp();
        int accepted = -1;
        for (int c = cur + 1; c < n; ++c) {
            if (sh.par[c] != cur) continue;
            const int x = sh.tok[c];
            // position of token x among the kept ones, or -1
            const uint32_t h0 = __ballot_sync(0xffffffffu, lane < m && sh.ktok[lane] == x);
            const uint32_t h1 = __ballot_sync(0xffffffffu, lane + 32 < m && sh.ktok[min(lane + 32, kMaxTopK - 1)] == x);
            const int jx = h0 ? __ffs(h0) - 1 : (h1 ? 31 + __ffs(h1) : -1);
            const double px = jx >= 0 ? sh.kp[jx] : 0.0;
            bool gone = jx >= 0 && sh.kgone[jx];
            if (jx < 0)  // a token outside the kept set may have been rejected here before (duplicate siblings)
                for (int c2 = cur + 1; c2 < c; ++c2) gone = gone || (sh.par[c2] == cur && sh.tok[c2] == x);
            const double qx = gone ? 0.0 : sh.tq0[c] * qscale;
            double ratio;
            if (qx > 0.0)
                ratio = px / qx;
            else
                ratio = px > 0.0 ? (double)INFINITY : 0.0;
            const double u = (double)sh.uni[c];
            if (lane == 0 && near_tie && fabs(ratio - u) < 1e-6) near_tie[(size_t)b * T + c] = 1;
            if (u < (ratio < 1.0 ? ratio : 1.0)) {
                accepted = c;
                break;
            }
            // rejected: the target becomes the normalised residual (over the kept tokens: everywhere else it is zero and
            // stays zero), the token leaves the draft distribution, which is renormalised
            double r0 = 0.0, r1 = 0.0;
            if (lane < m) r0 = fmax(sh.kp[lane] - (sh.kgone[lane] ? 0.0 : sh.kq0[lane] * qscale), 0.0);
            if (lane + 32 < m) r1 = fmax(sh.kp[lane + 32] - (sh.kgone[lane + 32] ? 0.0 : sh.kq0[lane + 32] * qscale), 0.0);
            double Z = r0 + r1;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) Z += __shfl_xor_sync(0xffffffffu, Z, o);
            __syncwarp();
            if (Z > 0.0) {
                if (lane < m) sh.kp[lane] = r0 / Z;
                if (lane + 32 < m) sh.kp[lane + 32] = r1 / Z;
            }
            if (lane == 0 && jx >= 0) sh.kgone[jx] = 1;
            __syncwarp();
            const double s = qtot - qx;  // mass left once x is gone
            if (!(s > 0.0)) break;
            qscale /= s;
            qtot = s / s;
        }
        if (accepted >= 0) {
            cur = accepted;
            __syncwarp();
            continue;
        }
        // final token: inverse CDF over the current target in vocabulary order (only kept tokens carry mass)
        for (int j = lane; j < m; j += 32) {
            int pos = 0;
            for (int i = 0; i < m; ++i) pos += sh.ktok[i] < sh.ktok[j] ? 1 : 0;
            sh.order[pos] = j;
        }
        __syncwarp();
        if (lane == 0) {
            double tot = 0.0;
            for (int i = 0; i < m; ++i) tot += sh.kp[sh.order[i]];
            const double target = (double)sh.uni[0] * tot;
            double run = 0.0;
            int pick = -1, last = sh.ktok[sh.order[0]];
            for (int i = 0; i < m; ++i) {
                const int j = sh.order[i];
                if (sh.kp[j] > 0.0) last = sh.ktok[j];
                run += sh.kp[j];
                if (run > target) {
                    pick = sh.ktok[j];
                    break;
                }
            }
            next_token[b] = pick >= 0 ? pick : last;
            for (int j = 0; j <= max_depth; ++j) pth[j] = -1;
            for (int t = cur; t >= 0; t = sh.par[t]) pth[sh.depth[t]] = t;
            accept_len[b] = sh.depth[cur];
        }
        return;
    }
}

// The selection kernel's grid: all rows' batches in equal runs, one CTA per run, about as many CTAs as the GPU holds at
// once (148 SMs x 3 CTAs of this kernel).  per: batches per CTA; pmax: most pieces (CTAs) that meet one row.
constexpr int kFsGridCtas = 148 * 3;
static inline void fs_split(int B, int T, int V, int* per, int* grid, int* pmax) {
    const long long nb = ceil_div(V, kFsSeg), total = nb * B * T;
    const long long ctas = std::min<long long>(total, kFsGridCtas);
    *per = (int)((total + ctas - 1) / ctas);
    *grid = (int)((total + *per - 1) / *per);
    *pmax = (int)((nb + *per - 1) / *per) + 1;
}
static inline size_t filtered_ws_layout(int B, int T, int V, int k, char* base, FCand** cand, double** qpart, KeptLists* kept) {
    size_t off = 0;
    const size_t rows = (size_t)B * T;
    int per, grid, P;
    fs_split(B, T, V, &per, &grid, &P);
    if (cand) *cand = reinterpret_cast<FCand*>(base + off);
    off += round_up(rows * P * k * sizeof(FCand), 256);
    if (qpart) *qpart = reinterpret_cast<double*>(base + off);
    off += round_up(rows * P * sizeof(double), 256);
    if (kept) kept->p = reinterpret_cast<double*>(base + off);
    off += round_up(rows * k * sizeof(double), 256);
    if (kept) kept->qtot = reinterpret_cast<double*>(base + off);
    off += round_up(rows * sizeof(double), 256);
    if (kept) kept->tok = reinterpret_cast<int32_t*>(base + off);
    off += round_up(rows * k * sizeof(int32_t), 256);
    if (kept) kept->q0 = reinterpret_cast<float*>(base + off);
    off += round_up(rows * k * sizeof(float), 256);
    if (kept) kept->n = reinterpret_cast<int32_t*>(base + off);
    off += round_up(rows * sizeof(int32_t), 256);
    return off;
}

}  // namespace s4c

extern "C" size_t s4c_tree_accept_filtered_workspace_bytes(int B, int T, int V, int top_k) {
    if (B < 1 || T < 1 || V < 1 || top_k < 1 || top_k > s4c::kMaxTopK) return 0;
    return s4c::filtered_ws_layout(B, T, V, top_k < V ? top_k : V, nullptr, nullptr, nullptr, nullptr);
}

extern "C" s4c_status s4c_tree_accept_filtered(const float* target_logits, const float* draft_probs, const int32_t* tokens,
                                               const int32_t* parent, const int32_t* n_nodes, float temperature,
                                               int top_k, float top_p, const float* uniforms, int B, int T, int V,
                                               int max_depth, int32_t* accept_len, int32_t* path, int32_t* next_token,
                                               uint8_t* near_tie, int32_t* status, void* workspace,
                                               size_t workspace_bytes, s4c_stream_t stream_) {
    using namespace s4c;
    if (!target_logits || !draft_probs || !tokens || !parent || !uniforms || !accept_len || !path || !next_token) return S4C_ERR_NULL;
    if (!(temperature > 0.f) || isinf(temperature)) return S4C_ERR_SHAPE;
    if (top_k < 1 || top_k > kMaxTopK || !(top_p > 0.f && top_p <= 1.f)) return S4C_ERR_SHAPE;
    if (B < 0 || B > 65535 || T < 1 || T > S4C_MAX_T || V < 1 || max_depth < 0 || max_depth >= S4C_MAX_T) return S4C_ERR_SHAPE;
    if (!aligned16(target_logits) || !aligned16(draft_probs)) return S4C_ERR_ALIGN;
    if (B == 0) return S4C_OK;
    const int k = top_k < V ? top_k : V;
    const size_t need = filtered_ws_layout(B, T, V, k, nullptr, nullptr, nullptr, nullptr);
    if (!workspace || workspace_bytes < need || !aligned256(workspace)) return S4C_ERR_WORKSPACE;
    FCand* cand;
    double* qpart;
    KeptLists kept;
    filtered_ws_layout(B, T, V, k, static_cast<char*>(workspace), &cand, &qpart, &kept);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int per, grid, pmax;
    fs_split(B, T, V, &per, &grid, &pmax);
    int G = kFsThreads;  // threads per group of the first threshold: the largest power of two with 256 / G >= k
    while (kFsThreads / G < k) G >>= 1;
    if (V % 4 == 0)
        filter_span_kernel<true><<<grid, kFsThreads, 0, stream>>>(target_logits, draft_probs, n_nodes, B * T, T, V, k, G, per, pmax,
                                                                  cand, qpart);
    else
        filter_span_kernel<false><<<grid, kFsThreads, 0, stream>>>(target_logits, draft_probs, n_nodes, B * T, T, V, k, G, per,
                                                                   pmax, cand, qpart);
    S4C_RETURN_IF_CUDA_ERROR();
    // the two kernels that follow are launched programmatically dependent: they become resident while their
    // predecessor drains and wait for its completion (griddepcontrol.wait) before they read what it wrote
    cudaLaunchAttribute pdl;
    pdl.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.stream = stream, cfg.attrs = &pdl, cfg.numAttrs = 1;
    cfg.gridDim = dim3(T, B, 1), cfg.blockDim = dim3(kFrThreads, 1, 1);
    if (cudaLaunchKernelEx(&cfg, filter_rows_kernel, (const FCand*)cand, (const double*)qpart, draft_probs, n_nodes, T, V, per,
                           pmax, k, 1.0 / (double)temperature, (double)top_p, kept) != cudaSuccess) {
        cudaGetLastError();
        return S4C_ERR_CUDA;
    }
    cfg.gridDim = dim3(B, 1, 1), cfg.blockDim = dim3(kFsThreads, 1, 1);
    if (cudaLaunchKernelEx(&cfg, accept_walk_sparse_kernel, draft_probs, tokens, parent, n_nodes, uniforms, T, V, k, max_depth,
                           kept, accept_len, path, next_token, near_tie, status) != cudaSuccess) {
        cudaGetLastError();
        return S4C_ERR_CUDA;
    }
    return S4C_OK;
}
