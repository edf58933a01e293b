// s4c_tree_accept_filtered: speculative-sampling acceptance (Section 2; Eq. 11, Eq. 12; longest accepted path,
// Section 3.2) against a top-k / nucleus FILTERED target distribution -- the sampling regime of Section 4 (RQ5).
//
// Filtering makes the target distribution sparse: at most top_k (<= 64) tokens per node keep any mass.  So the only
// vocabulary-wide work is finding those tokens, a selection over the logits that needs no exponential at all:
//   filter_segments_kernel  grid (vocabulary segments of 4096, T, B): every thread sorts its 16 logits (with their token
//                           indices, order: logit descending, token ascending), every warp merges its lanes' sorted lists
//                           head by head into its k best, one warp merges the eight warp lists into the segment's k best
//   filter_rows_kernel      grid (T, B), one warp: merges the segments' lists into the row's k best, turns them into
//                           probabilities in float64 (softmax over the kept logits at the temperature), cuts the nucleus
//                           and renormalises: per node a short list (token, probability) in rank order
//   accept_walk_sparse_kernel  grid (B): the walk of s4c_tree_accept on these lists.  Residual masses and the final
//                           inverse-CDF draw run over the <= 64 kept tokens of a node; only the renormalisation of the
//                           draft distribution after a rejection needs its sum over the vocabulary, one CTA-wide pass
//                           over the draft row of that node.
// HBM traffic: every logits row once (the draft rows only where a rejection happens).  Ranking, sums and decisions are
// deterministic (fixed orders); ties between equal logits go to the lower token.
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

template <bool VEC>
__global__ void __launch_bounds__(kFsThreads)
filter_segments_kernel(const float* __restrict__ logits, const int32_t* __restrict__ n_nodes, int T, int V, int k,
                       FCand* __restrict__ cand) {
    const int seg = blockIdx.x, node = blockIdx.y, b = blockIdx.z;
    if (n_nodes && node >= n_nodes[b]) return;
    const float* row = logits + ((size_t)b * T + node) * V;
    const int s0 = seg * kFsSeg, tid = threadIdx.x, warp = tid >> 5;
    float x[kFsElems];
    int e[kFsElems];
#pragma unroll
    for (int i = 0; i < kFsElems; ++i) e[i] = VEC ? s0 + ((i >> 2) * kFsThreads + tid) * 4 + (i & 3) : s0 + i * kFsThreads + tid;
    if (VEC) {
#pragma unroll
        for (int i = 0; i < kFsElems / 4; ++i) {
            float4 v = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
            if (e[4 * i] < V) v = __ldg(reinterpret_cast<const float4*>(row + e[4 * i]));  // V % 4 == 0 here
            x[4 * i + 0] = v.x, x[4 * i + 1] = v.y, x[4 * i + 2] = v.z, x[4 * i + 3] = v.w;
        }
    } else {
#pragma unroll
        for (int i = 0; i < kFsElems; ++i) x[i] = e[i] < V ? __ldg(row + e[i]) : -INFINITY;
    }
    // a NaN or +Inf anywhere in the segment: the row is unusable (the walk flags the sequence); say so in the first slot
    float mx = x[0];
#pragma unroll
    for (int i = 1; i < kFsElems; ++i) mx = fmax_keep_nan(mx, x[i]);
    const int bad = __syncthreads_or(!(mx < INFINITY));
    FCand* out = cand + (((size_t)b * T + node) * gridDim.x + seg) * k;
    if (bad) {
        for (int r = tid; r < k; r += kFsThreads) out[r].x = r == 0 ? INFINITY : -INFINITY, out[r].tok = r == 0 ? 0 : INT_MAX;
        return;
    }
#pragma unroll
    for (int i = 0; i < kFsElems; ++i)
        if (e[i] >= V) e[i] = INT_MAX;  // entries beyond the row rank last
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
    __shared__ FCand lists[kFsElems][kFsThreads];       // entry h of thread t at [h][t]
    __shared__ FCand wlist[kFsThreads / 32][kMaxTopK];  // the warps' k best
#pragma unroll
    for (int i = 0; i < kFsElems; ++i) lists[i][tid].x = x[i], lists[i][tid].tok = e[i];
    __syncwarp();
    merge_heads(&lists[0][warp * 32], 32, kFsElems, kFsThreads, 1, k, wlist[warp]);
    __syncthreads();
    if (warp == 0) merge_heads(&wlist[0][0], kFsThreads / 32, k, 1, kMaxTopK, k, out);
}

struct KeptLists {  // per (sequence, node): the filtered target distribution
    int32_t* n;     // [B*T]: kept tokens (1..top_k); -1: the row is unusable (NaN / +Inf logit, or nothing but -Inf)
    int32_t* tok;   // [B*T*k] in rank order
    double* p;      // [B*T*k]
};

__global__ void __launch_bounds__(32)
filter_rows_kernel(const FCand* __restrict__ cand, const int32_t* __restrict__ n_nodes, int T, int segs, int k, double inv_tau,
                   double top_p, KeptLists kept) {
    const int node = blockIdx.x, b = blockIdx.y, lane = threadIdx.x;
    if (n_nodes && node >= n_nodes[b]) return;
    __shared__ FCand best[2][kMaxTopK];
    __shared__ FCand stage[32][kMaxTopK];
    const FCand* c = cand + ((size_t)b * T + node) * segs * k;
    // the row's k best out of the segments' lists: 31 lists at a time, each round merged with the best so far
    int have = 0, cur = 0;
    for (int s0 = 0; s0 < segs; s0 += 31) {
        const int ns = min(31, segs - s0);
        for (int i = lane; i < ns * k; i += 32) stage[i / k][i % k] = c[(size_t)(s0 + i / k) * k + i % k];
        if (have)
            for (int i = lane; i < k; i += 32) stage[ns][i] = best[cur][i];
        __syncwarp();
        merge_heads(&stage[0][0], ns + (have ? 1 : 0), k, 1, kMaxTopK, k, best[cur ^ 1]);
        __syncwarp();
        cur ^= 1, have = 1;
    }
    const FCand* top = best[cur];
    const size_t at = (size_t)b * T + node;
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
    }
    __syncwarp();
    for (int j = lane; j < k; j += 32) {
        kept.tok[at * k + j] = j < m_s ? top[j].tok : -1;
        kept.p[at * k + j] = j < m_s ? ej[j] / mass_s : 0.0;
    }
}

struct SparseShared {
    int32_t par[S4C_MAX_T];
    int32_t tok[S4C_MAX_T];
    float uni[S4C_MAX_T];
    int depth[S4C_MAX_T];
    uint32_t anc[S4C_MAX_T][S4C_MASK_WORDS];
    double tq0[S4C_MAX_T];   // draft probability of node i's token under its parent's row
    int ktok[kMaxTopK];      // the current node's kept tokens, in TOKEN order (the order the vocabulary is scanned in)
    double kp[kMaxTopK];     // their current target probabilities
    double kq0[kMaxTopK];    // their draft probabilities as given
    int kgone[kMaxTopK];     // 1: the token was rejected here and has left the draft distribution
    double red[kFsThreads / 32];
    int flag;
};

__global__ void __launch_bounds__(kFsThreads)
accept_walk_sparse_kernel(const float* __restrict__ dprobs, const int32_t* __restrict__ tokens, const int32_t* __restrict__ parent,
                          const int32_t* __restrict__ n_nodes, const float* __restrict__ uniforms, int T, int V, int k,
                          int max_depth, KeptLists kept, int32_t* __restrict__ accept_len, int32_t* __restrict__ path,
                          int32_t* __restrict__ next_token, uint8_t* __restrict__ near_tie, int32_t* __restrict__ status) {
    __shared__ SparseShared sh;
    const int b = blockIdx.x, tid = threadIdx.x;
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

    int cur = 0;
    for (int guard = 0; guard <= T; ++guard) {
        const size_t at = (size_t)b * T + cur;
        const float* qrow = dprobs + at * V;
        const int m = kept.n[at];
        // the kept tokens in token order: entry j goes to the position given by the number of smaller tokens
        if (tid < m) {
            const int t = kept.tok[at * k + tid];
            int pos = 0;
            for (int j = 0; j < m; ++j) pos += kept.tok[at * k + j] < t ? 1 : 0;
            sh.ktok[pos] = t, sh.kp[pos] = kept.p[at * k + tid], sh.kq0[pos] = (double)__ldg(qrow + t), sh.kgone[pos] = 0;
        }
        __syncthreads();
        auto find = [&](int x) {  // position of token x among the kept ones, or -1
            for (int j = 0; j < m; ++j)
                if (sh.ktok[j] == x) return j;
            return -1;
        };
        double qscale = 1.0;   // the draft distribution is the given row times this, rejected tokens left out
        double qtot = 0.0;     // its total mass (computed when the first rejection needs it)
        bool have_qtot = false;
        int accepted = -1;
        for (int c = cur + 1; c < n; ++c) {
            if (sh.par[c] != cur) continue;
            const int x = sh.tok[c];
            const int jx = find(x);
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
            if (tid == 0 && near_tie && fabs(ratio - u) < 1e-6) near_tie[(size_t)b * T + c] = 1;
            if (u < (ratio < 1.0 ? ratio : 1.0)) {
                accepted = c;
                break;
            }
            // rejected: the target becomes the normalised residual (over the kept tokens: everywhere else it is zero and
            // stays zero), the token leaves the draft distribution, which is renormalised
            if (!have_qtot) {  // the draft row's mass: one pass of the CTA over the row, fixed order
                double part = 0.0;
                for (int v = tid; v < V; v += blockDim.x) part += (double)__ldg(qrow + v);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                __syncthreads();
                if ((tid & 31) == 0) sh.red[tid >> 5] = part;
                __syncthreads();
                qtot = 0.0;
                for (int w = 0; w < kFsThreads / 32; ++w) qtot += sh.red[w];
                have_qtot = true;
            }
            __syncthreads();  // everyone has read the lists before thread 0 rewrites them
            if (tid == 0) {
                double Z = 0.0;
                for (int j = 0; j < m; ++j) {
                    const double r = sh.kp[j] - (sh.kgone[j] ? 0.0 : sh.kq0[j] * qscale);
                    Z += r > 0.0 ? r : 0.0;
                }
                if (Z > 0.0)
                    for (int j = 0; j < m; ++j) {
                        const double r = sh.kp[j] - (sh.kgone[j] ? 0.0 : sh.kq0[j] * qscale);
                        sh.kp[j] = r > 0.0 ? r / Z : 0.0;
                    }
                if (jx >= 0) sh.kgone[jx] = 1;
            }
            __syncthreads();
            const double s = qtot - qx;  // mass left once x is gone
            if (!(s > 0.0)) break;
            qscale /= s;
            qtot = s / s;
        }
        if (accepted >= 0) {
            cur = accepted;
            __syncthreads();
            continue;
        }
        // final token: inverse CDF over the current target in vocabulary order (only kept tokens carry mass)
        if (tid == 0) {
            double tot = 0.0;
            for (int j = 0; j < m; ++j) tot += sh.kp[j];
            const double target = (double)sh.uni[0] * tot;
            double run = 0.0;
            int pick = -1, last = sh.ktok[0];
            for (int j = 0; j < m; ++j) {
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
static inline size_t filtered_ws_layout(int B, int T, int V, int k, char* base, FCand** cand, KeptLists* kept) {
    size_t off = 0;
    if (cand) *cand = reinterpret_cast<FCand*>(base + off);
    off += round_up((size_t)B * T * fs_segments(V) * k * sizeof(FCand), 256);
    if (kept) kept->p = reinterpret_cast<double*>(base + off);
    off += round_up((size_t)B * T * k * sizeof(double), 256);
    if (kept) kept->tok = reinterpret_cast<int32_t*>(base + off);
    off += round_up((size_t)B * T * k * sizeof(int32_t), 256);
    if (kept) kept->n = reinterpret_cast<int32_t*>(base + off);
    off += round_up((size_t)B * T * sizeof(int32_t), 256);
    return off;
}

}  // namespace s4c

extern "C" size_t s4c_tree_accept_filtered_workspace_bytes(int B, int T, int V, int top_k) {
    if (B < 1 || T < 1 || V < 1 || top_k < 1 || top_k > s4c::kMaxTopK) return 0;
    return s4c::filtered_ws_layout(B, T, V, top_k < V ? top_k : V, nullptr, nullptr, nullptr);
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
    const size_t need = filtered_ws_layout(B, T, V, k, nullptr, nullptr, nullptr);
    if (!workspace || workspace_bytes < need || !aligned256(workspace)) return S4C_ERR_WORKSPACE;
    FCand* cand;
    KeptLists kept;
    filtered_ws_layout(B, T, V, k, static_cast<char*>(workspace), &cand, &kept);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int segs = fs_segments(V);
    dim3 grid(segs, T, B);
    if (V % 4 == 0)
        filter_segments_kernel<true><<<grid, kFsThreads, 0, stream>>>(target_logits, n_nodes, T, V, k, cand);
    else
        filter_segments_kernel<false><<<grid, kFsThreads, 0, stream>>>(target_logits, n_nodes, T, V, k, cand);
    S4C_RETURN_IF_CUDA_ERROR();
    filter_rows_kernel<<<dim3(T, B), 32, 0, stream>>>(cand, n_nodes, T, segs, k, 1.0 / (double)temperature, (double)top_p, kept);
    S4C_RETURN_IF_CUDA_ERROR();
    accept_walk_sparse_kernel<<<B, kFsThreads, 0, stream>>>(draft_probs, tokens, parent, n_nodes, uniforms, T, V, k, max_depth,
                                                            kept, accept_len, path, next_token, near_tie, status);
    S4C_RETURN_IF_CUDA_ERROR();
    return S4C_OK;
}
