// s4c_tree_accept_filtered: speculative-sampling acceptance (Section 2; Eq. 11, Eq. 12; longest accepted path,
// Section 3.2) against a top-k / nucleus FILTERED target distribution -- the sampling regime of Section 4 (RQ5).
//
// Filtering makes the target distribution sparse: at most top_k (<= 64) tokens per node keep any mass.  So the only
// vocabulary-wide work is finding those tokens -- a selection over the logits that needs no exponential -- and the mass
// of every draft row (the renormalisation after a rejection needs it):
//   filter_segments_kernel  grid (vocabulary segments of 4096, T, B), one pass over logits and draft probabilities:
//                           the segment's k best logits by THRESHOLD SELECTION.  The k-th best of the segment is at
//                           least the smallest of the 256 threads' maxima, so only entries at or above that value
//                           matter (about a third of them); these are counted in a 256-bin histogram over
//                           [that value, the segment's maximum], the bin where the count from the top reaches k is
//                           found, the entries of the bins down to it (k plus a few) are gathered and ranked exactly
//                           (logit descending, token ascending) by counting.  Segments that this cannot serve (more
//                           than 256 entries in those bins: heavy ties; fewer than k threads with a finite logit) take
//                           a slower exact path: every thread sorts its 16 entries, warps merge their lanes' lists head
//                           by head, one warp merges the warps' lists.  Also the segment's draft mass in float64.
//   filter_rows_kernel      grid (T, B): merges the segments' sorted lists pairwise (a bitonic merge of two lists in a
//                           warp's registers, a tree of such merges over the lists) into the row's k best, turns them
//                           into probabilities in float64 (softmax over the kept logits at the temperature), cuts the
//                           nucleus and renormalises: per node a short list (token, probability, draft probability) in
//                           rank order, and the draft row's mass
//   accept_walk_sparse_kernel  grid (B): the walk of s4c_tree_accept on these lists, by one warp: acceptance tests,
//                           residual masses and the final inverse-CDF draw run over the <= 64 kept tokens of a node.
// HBM traffic: every logits row and every draft row once.  Ranking, sums and decisions are deterministic (fixed orders);
// ties between equal logits go to the lower token.
#include <float.h>
#include <limits.h>
#include <math.h>

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
constexpr uint32_t kKeyPosInf = 0xff800000u;  // f_key(+inf)
constexpr uint32_t kKeyNegInf = 0x007fffffu;  // f_key(-inf)

constexpr int kFsBins = 256;   // histogram bins of the threshold selection
constexpr int kFsCap = 256;    // most candidates ranked by counting (one per thread)

struct SegShared {
    union {
        struct {
            FCand lists[kFsElems][kFsThreads];       // slow path: entry h of thread t at [h][t]
            FCand wlist[kFsThreads / 32][kMaxTopK];  // slow path: the warps' k best
        } slow;
        struct {
            int hist[kFsBins];
            FCand cand[kFsCap];
        } fast;
    };
    uint32_t wmax[kFsThreads / 32], wmin[kFsThreads / 32];
    int wfin[kFsThreads / 32];
    double wq[kFsThreads / 32];
    int ncand;
};

template <bool VEC>
__global__ void __launch_bounds__(kFsThreads)
filter_segments_kernel(const float* __restrict__ logits, const float* __restrict__ dprobs, const int32_t* __restrict__ n_nodes,
                       int T, int V, int k, FCand* __restrict__ cand, double* __restrict__ qpart) {
    const int seg = blockIdx.x, node = blockIdx.y, b = blockIdx.z;
    if (n_nodes && node >= n_nodes[b]) return;
    __shared__ SegShared sh;
    const size_t at = (size_t)b * T + node;
    const float* row = logits + at * V;
    const float* qrow = dprobs + at * V;
    const int s0 = seg * kFsSeg, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // entry i of this thread is token tok_of(i); the same map on every path
    auto tok_of = [&](int i) { return VEC ? s0 + ((i >> 2) * kFsThreads + tid) * 4 + (i & 3) : s0 + i * kFsThreads + tid; };
    float x[kFsElems];
    double qs = 0.0;
    if (VEC) {  // V % 4 == 0: whole 16-byte words, all requested before any is used
        float4 lv[kFsElems / 4], qv[kFsElems / 4];
#pragma unroll
        for (int i = 0; i < kFsElems / 4; ++i) {
            lv[i] = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY), qv[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (tok_of(4 * i) < V) {
                lv[i] = __ldg(reinterpret_cast<const float4*>(row + tok_of(4 * i)));
                qv[i] = __ldg(reinterpret_cast<const float4*>(qrow + tok_of(4 * i)));
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
            const bool in = tok_of(i) < V;
            x[i] = in ? __ldg(row + tok_of(i)) : -INFINITY;
            q[i] = in ? __ldg(qrow + tok_of(i)) : 0.f;
        }
#pragma unroll
        for (int i = 0; i < kFsElems; ++i) qs += (double)q[i];
    }
    // the thread's maximum (a NaN survives), then per warp: the largest and the smallest finite thread maximum and how
    // many threads have a finite one; the warp's draft mass
    float mx = x[0];
#pragma unroll
    for (int i = 1; i < kFsElems; ++i) mx = fmax_keep_nan(mx, x[i]);
    const uint32_t key = mx < INFINITY ? f_key(mx) : 0xffffffffu;  // NaN (whatever its bits) and +Inf rank on top
    const bool fin = key > kKeyNegInf;  // the thread holds something above -inf
    const uint32_t kmax = __reduce_max_sync(0xffffffffu, key);
    const uint32_t kmin = __reduce_min_sync(0xffffffffu, fin ? key : 0xffffffffu);
    const int nfin_w = __popc(__ballot_sync(0xffffffffu, fin));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) qs += __shfl_xor_sync(0xffffffffu, qs, o);
    if (lane == 0) sh.wmax[warp] = kmax, sh.wmin[warp] = kmin, sh.wfin[warp] = nfin_w, sh.wq[warp] = qs;
    sh.fast.hist[tid] = 0;  // kFsBins == kFsThreads
    if (tid == 0) sh.ncand = 0;
    __syncthreads();
    uint32_t Kmax = 0, Kmin = 0xffffffffu;
    int n_fin = 0;
#pragma unroll
    for (int w = 0; w < kFsThreads / 32; ++w) Kmax = max(Kmax, sh.wmax[w]), Kmin = min(Kmin, sh.wmin[w]), n_fin += sh.wfin[w];
    if (tid == 0) {
        double tot = 0.0;
        for (int w = 0; w < kFsThreads / 32; ++w) tot += sh.wq[w];
        qpart[at * gridDim.x + seg] = tot;
    }
    FCand* out = cand + (at * gridDim.x + seg) * k;
    if (Kmax >= kKeyPosInf) {  // a NaN or +Inf in the segment: the row is unusable (the walk flags the sequence)
        for (int r = tid; r < k; r += kFsThreads) out[r].x = r == 0 ? INFINITY : -INFINITY, out[r].tok = r == 0 ? 0 : INT_MAX;
        return;
    }
    const int n_valid = min(kFsSeg, V - s0);
    // ---- which entries can be among the k best (CTA-uniform decisions)
    int n_cand = -1;  // -1: the slow path
    if (n_valid <= kFsCap) {  // a short tail segment: every entry is a candidate
#pragma unroll
        for (int i = 0; i < kFsElems; ++i)
            if (tok_of(i) < V) {
                const int slot = atomicAdd(&sh.ncand, 1);
                sh.fast.cand[slot].x = x[i], sh.fast.cand[slot].tok = tok_of(i);
            }
        n_cand = n_valid;
    } else if (n_fin >= k) {
        // at least n_fin >= k entries are >= lo, so nothing below lo is among the k best; bins fall with the logit
        // (float subtraction, multiplication by a positive constant and truncation are monotone), equal logits share a bin
        const float M = f_unkey(Kmax), lo = f_unkey(Kmin);
        const float inv = (float)kFsBins / (M - lo);
        auto bin_of = [&](float v) { return min(kFsBins - 1, (int)((M - v) * inv)); };  // (int)NaN = 0: M == lo
#pragma unroll
        for (int i = 0; i < kFsElems; ++i)
            if (x[i] >= lo) atomicAdd(&sh.fast.hist[bin_of(x[i])], 1);
        __syncthreads();
        // every warp finds the bin where the count from the top reaches k (the same scan in every warp: no broadcast)
        int c8[8], mine = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) c8[j] = sh.fast.hist[lane * 8 + j], mine += c8[j];
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        const uint32_t reach = __ballot_sync(0xffffffffu, incl >= k);  // not empty: the bins hold >= n_fin >= k entries
        const int L = __ffs(reach) - 1;
        int bstar = 0, ctot = 0;
        if (lane == L) {
            int run = incl - mine;
            for (int j = 0; j < 8; ++j) {
                run += c8[j];
                if (run >= k) {
                    bstar = lane * 8 + j, ctot = run;
                    break;
                }
            }
        }
        bstar = __shfl_sync(0xffffffffu, bstar, L), ctot = __shfl_sync(0xffffffffu, ctot, L);
        if (ctot <= kFsCap) {
#pragma unroll
            for (int i = 0; i < kFsElems; ++i)
                if (x[i] >= lo && bin_of(x[i]) <= bstar) {
                    const int slot = atomicAdd(&sh.ncand, 1);
                    sh.fast.cand[slot].x = x[i], sh.fast.cand[slot].tok = tok_of(i);
                }
            n_cand = ctot;
        }
    }
    __syncthreads();
    if (n_cand >= 0) {
        // exact ranks among the candidates by counting; the order is total, so the ranks are 0 .. n_cand-1
        if (tid < n_cand) {
            const FCand me = sh.fast.cand[tid];
            int r = 0;
            for (int j = 0; j < n_cand; ++j) {
                const FCand o = sh.fast.cand[j];
                r += f_before(o.x, o.tok, me.x, me.tok) ? 1 : 0;
            }
            if (r < k) out[r] = me;
        }
        for (int r = n_cand + tid; r < k; r += kFsThreads) out[r].x = -INFINITY, out[r].tok = INT_MAX;
        return;
    }
    // ---- the slow exact path (the barrier above: nobody reads the histogram any more, its memory is reused)
    int e[kFsElems];
#pragma unroll
    for (int i = 0; i < kFsElems; ++i) e[i] = tok_of(i) < V ? tok_of(i) : INT_MAX;  // entries beyond the row rank last
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
    for (int i = 0; i < kFsElems; ++i) sh.slow.lists[i][tid].x = x[i], sh.slow.lists[i][tid].tok = e[i];
    __syncwarp();
    merge_heads(&sh.slow.lists[0][warp * 32], 32, kFsElems, kFsThreads, 1, k, sh.slow.wlist[warp]);
    __syncthreads();
    if (warp == 0) merge_heads(&sh.slow.wlist[0][0], kFsThreads / 32, k, 1, kMaxTopK, k, out);
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
                   const int32_t* __restrict__ n_nodes, int T, int V, int segs, int k, double inv_tau, double top_p,
                   KeptLists kept) {
    const int node = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (n_nodes && node >= n_nodes[b]) return;
    __shared__ FCand A[kFrLists][kMaxTopK];
    const size_t at = (size_t)b * T + node;
    const FCand* c = cand + at * segs * k;
    // the row's best out of the segments' lists: 32 lists at a time (later rounds: the best so far and 31 new ones),
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
    __shared__ int m_s;
    __shared__ double mass_s;
    if (lane == 0) {
        int kk = 0;
        while (kk < k && top[kk].tok != INT_MAX) ++kk;  // (fewer than k tokens in the vocabulary)
        double mass = 0.0;
        for (int j = 0; j < kk; ++j) mass += ej[j];
        int m = kk;
        if (top_p < 1.0) {
            double cum = 0.0;
            for (int j = 0; j < kk; ++j) {
                cum += ej[j] / mass;
                if (cum >= top_p) {
                    m = j + 1;
                    break;
                }
            }
            mass = 0.0;
            for (int j = 0; j < m; ++j) mass += ej[j];
        }
        m_s = m, mass_s = mass;
        kept.n[at] = m;
        double qt = 0.0;  // the draft row's mass: the segments' sums in segment order
        for (int s = 0; s < segs; ++s) qt += qpart[at * segs + s];
        kept.qtot[at] = qt;
    }
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
            if (kept.n[(size_t)b * T + i] < 0) atomicOr(&sh.flag, S4C_SEQ_NONFINITE);
        }
        __syncthreads();
        flags = sh.flag;
    }
    if (tid == 0 && status) status[b] = flags;
    if (flags) {
        for (int j = tid; j <= max_depth; j += blockDim.x) pth[j] = -1;
        if (tid == 0) accept_len[b] = -1, next_token[b] = -1;
        return;
    }
    for (int i = 1 + tid; i < n; i += blockDim.x)
        sh.tq0[i] = (double)__ldg(dprobs + ((size_t)b * T + sh.par[i]) * V + sh.tok[i]);
    __syncthreads();
    if (tid >= 32) return;  // the walk itself is one warp's work: lists of at most 64 entries, two per lane

    int cur = 0;
    for (int guard = 0; guard <= T; ++guard) {
        const size_t at = (size_t)b * T + cur;
        const int m = kept.n[at];
        double qtot = kept.qtot[at];  // mass of the draft distribution as it stands
        double qscale = 1.0;          // the draft distribution is the given row times this, rejected tokens left out
        for (int j = lane; j < m; j += 32)
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

static inline int fs_segments(int V) { return ceil_div(V, kFsSeg); }
static inline size_t filtered_ws_layout(int B, int T, int V, int k, char* base, FCand** cand, double** qpart, KeptLists* kept) {
    size_t off = 0;
    const size_t rows = (size_t)B * T;
    if (cand) *cand = reinterpret_cast<FCand*>(base + off);
    off += round_up(rows * fs_segments(V) * k * sizeof(FCand), 256);
    if (qpart) *qpart = reinterpret_cast<double*>(base + off);
    off += round_up(rows * fs_segments(V) * sizeof(double), 256);
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
    const int segs = fs_segments(V);
    dim3 grid(segs, T, B);
    if (V % 4 == 0)
        filter_segments_kernel<true><<<grid, kFsThreads, 0, stream>>>(target_logits, draft_probs, n_nodes, T, V, k, cand, qpart);
    else
        filter_segments_kernel<false><<<grid, kFsThreads, 0, stream>>>(target_logits, draft_probs, n_nodes, T, V, k, cand, qpart);
    S4C_RETURN_IF_CUDA_ERROR();
    filter_rows_kernel<<<dim3(T, B), kFrThreads, 0, stream>>>(cand, qpart, draft_probs, n_nodes, T, V, segs, k,
                                                              1.0 / (double)temperature, (double)top_p, kept);
    S4C_RETURN_IF_CUDA_ERROR();
    accept_walk_sparse_kernel<<<B, kFsThreads, 0, stream>>>(draft_probs, tokens, parent, n_nodes, uniforms, T, V, k, max_depth,
                                                            kept, accept_len, path, next_token, near_tie, status);
    S4C_RETURN_IF_CUDA_ERROR();
    return S4C_OK;
}
