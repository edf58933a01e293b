// s4c_tree_accept: acceptance of the draft tree against the target logits.
//   greedy (Section 4.1.2) and speculative sampling (Section 2; Eq. 11, Eq. 12), walked along
//   root-to-leaf paths to the longest accepted path (Section 3.2).
//
// Three kernels, all HBM-streaming or latency-bound, no tensor cores (there is no contraction here):
//   1. accept_rowstats_kernel   grid (vocab segments, T, B): every CTA holds one 4096-element segment of
//      one logits row in registers (16-byte coalesced loads), reduces (max, lowest argmax) with warp
//      shuffles and, for sampling, the segment's sum of exp((x - max_seg)/tau) in float64.
//   2. accept_residual_kernel   (sampling only) same grid: merges the row's segment statistics, then
//      streams the logits segment again (L2) with the draft-probability segment and reduces the
//      first-round residual mass  Z1 = sum max(p - q, 0)  and the draft mass left after removing the
//      first child's token -- what the walk needs after the first rejection at any node.
//   3. accept_walk_kernel       one CTA per sequence: validates the tree, merges per-node statistics,
//      walks root to leaf.  Second and later rejections at one node need a new residual mass; those
//      and the final inverse-CDF draw are CTA-wide passes over that single row.
// Every sum that feeds a decision is float64 with a fixed reduction order, so results do not depend on
// scheduling and agree with a sequential float64 evaluation to rounding (~1e-15 relative).
#include <float.h>
#include <math.h>

#include "s4c_common.cuh"

namespace s4c {

constexpr int kRowThreads = 256;
constexpr int kElemsPerThread = 16;
constexpr int kSegElems = kRowThreads * kElemsPerThread;  // 4096 logits per CTA
constexpr int kWalkThreads = 1024;

struct RowPartial {  // one vocab segment of one row
    double S;        // sum exp((x - M)/tau) over the segment (sampling only)
    float M;         // segment max
    int idx;         // lowest index attaining M
};
struct ResPartial {
    double Z;  // sum max(p - q, 0) over the segment
    double Q;  // sum of q over the segment, the first child's token left out
};
struct NodeStats {
    double S;
    float M;
    int idx;
};

static inline int accept_splits(int V) { return ceil_div(V, kSegElems); }

struct AcceptWorkspace {
    RowPartial* row;
    ResPartial* res;
    NodeStats* node;
};
static inline size_t accept_ws_layout(int B, int T, int V, char* base, AcceptWorkspace* ws) {
    const size_t n = (size_t)B * T * accept_splits(V);
    size_t off = 0;
    if (ws) ws->row = reinterpret_cast<RowPartial*>(base + off);
    off += round_up(n * sizeof(RowPartial), 256);
    if (ws) ws->res = reinterpret_cast<ResPartial*>(base + off);
    off += round_up(n * sizeof(ResPartial), 256);
    if (ws) ws->node = reinterpret_cast<NodeStats*>(base + off);
    off += round_up((size_t)B * T * sizeof(NodeStats), 256);
    return off;
}

// ----------------------------------------------------------------------------- reductions
__device__ __forceinline__ void argmax_combine(float& m, int& i, float om, int oi) {
    if (om > m || (om == m && oi < i)) {
        m = om;
        i = oi;
    }
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum over the CTA in a fixed order; result valid in every thread.  `scratch` holds >= 33 doubles.
__device__ __forceinline__ double block_sum(double v, double* scratch) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    v = warp_sum(v);
    __syncthreads();  // scratch may still be read from a previous call
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    if (warp == 0) {
        double t = lane < nwarps ? scratch[lane] : 0.0;
        t = warp_sum(t);
        if (lane == 0) scratch[32] = t;
    }
    __syncthreads();
    return scratch[32];
}

// ----------------------------------------------------------------------------- kernel 1
template <bool VEC>
__device__ __forceinline__ void load_segment(const float* __restrict__ row, int s0, int V, float (&x)[kElemsPerThread]) {
    if (VEC) {
#pragma unroll
        for (int k = 0; k < kElemsPerThread / 4; ++k) {
            const int e = s0 + (k * kRowThreads + threadIdx.x) * 4;
            float4 v = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
            if (e < V) v = __ldg(reinterpret_cast<const float4*>(row + e));  // V % 4 == 0 here
            x[4 * k + 0] = v.x, x[4 * k + 1] = v.y, x[4 * k + 2] = v.z, x[4 * k + 3] = v.w;
        }
    } else {
#pragma unroll
        for (int k = 0; k < kElemsPerThread; ++k) {
            const int e = s0 + k * kRowThreads + threadIdx.x;
            x[k] = e < V ? __ldg(row + e) : -INFINITY;
        }
    }
}
template <bool VEC>
__device__ __forceinline__ int elem_index(int s0, int k) {
    return VEC ? s0 + ((k >> 2) * kRowThreads + threadIdx.x) * 4 + (k & 3) : s0 + k * kRowThreads + threadIdx.x;
}

template <bool STOCH, bool VEC>
__global__ void __launch_bounds__(kRowThreads)
accept_rowstats_kernel(const float* __restrict__ logits, const int32_t* __restrict__ n_nodes, int T, int V,
                       double inv_tau, RowPartial* __restrict__ out) {
    const int split = blockIdx.x, node = blockIdx.y, b = blockIdx.z;
    if (n_nodes && node >= n_nodes[b]) return;
    const float* row = logits + ((size_t)b * T + node) * V;
    const int s0 = split * kSegElems;
    float x[kElemsPerThread];
    load_segment<VEC>(row, s0, V, x);

    float m = -INFINITY;
    int mi = INT_MAX;
#pragma unroll
    for (int k = 0; k < kElemsPerThread; ++k) {
        const int e = elem_index<VEC>(s0, k);
        if (e < V) argmax_combine(m, mi, x[k], e);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, m, o);
        const int oi = __shfl_xor_sync(0xffffffffu, mi, o);
        argmax_combine(m, mi, om, oi);
    }
    __shared__ float sm[kRowThreads / 32];
    __shared__ int si[kRowThreads / 32];
    __shared__ double scratch[33];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) sm[warp] = m, si[warp] = mi;
    __syncthreads();
    m = sm[0], mi = si[0];
#pragma unroll
    for (int w = 1; w < kRowThreads / 32; ++w) argmax_combine(m, mi, sm[w], si[w]);

    double S = 0.0;
    if (STOCH) {
        double s = 0.0;
        if (m > -INFINITY) {
            const double md = (double)m;
#pragma unroll
            for (int k = 0; k < kElemsPerThread; ++k) {
                const int e = elem_index<VEC>(s0, k);
                if (e < V) s += exp(((double)x[k] - md) * inv_tau);
            }
        }
        S = block_sum(s, scratch);
    }
    if (threadIdx.x == 0) {
        RowPartial r;
        r.S = S, r.M = m, r.idx = mi;
        out[((size_t)b * T + node) * gridDim.x + split] = r;
    }
}

// Merges the segment statistics of one row in split order: M = max, S = sum S_i exp((M_i - M)/tau).
__device__ __forceinline__ NodeStats merge_row(const RowPartial* __restrict__ part, int splits, double inv_tau,
                                               bool want_sum) {
    NodeStats r;
    r.M = -INFINITY, r.idx = INT_MAX, r.S = 0.0;
    for (int s = 0; s < splits; ++s) argmax_combine(r.M, r.idx, part[s].M, part[s].idx);
    if (want_sum && r.M > -INFINITY)
        for (int s = 0; s < splits; ++s)
            if (part[s].M > -INFINITY) r.S += part[s].S * exp(((double)part[s].M - (double)r.M) * inv_tau);
    return r;
}

// ----------------------------------------------------------------------------- kernel 2
template <bool VEC>
__global__ void __launch_bounds__(kRowThreads)
accept_residual_kernel(const float* __restrict__ logits, const float* __restrict__ dprobs,
                       const int32_t* __restrict__ tokens, const int32_t* __restrict__ parent,
                       const int32_t* __restrict__ n_nodes, int T, int V, double inv_tau,
                       const RowPartial* __restrict__ rowp, ResPartial* __restrict__ resp,
                       NodeStats* __restrict__ nodes) {
    const int split = blockIdx.x, node = blockIdx.y, b = blockIdx.z, splits = gridDim.x;
    const int n = n_nodes ? n_nodes[b] : T;
    if (node >= n || n > T) return;
    __shared__ NodeStats ns;
    __shared__ int first_tok;
    __shared__ double scratch[33];
    if (threadIdx.x == 0) {
        ns = merge_row(rowp + ((size_t)b * T + node) * splits, splits, inv_tau, true);
        if (split == 0) nodes[(size_t)b * T + node] = ns;
    }
    if (threadIdx.x == 32) {  // token of the first child in index order (the first one ever rejected here)
        int ft = -1;
        for (int c = node + 1; c < n; ++c)
            if (parent[(size_t)b * T + c] == node) {
                ft = tokens[(size_t)b * T + c];
                break;
            }
        first_tok = ft;
    }
    __syncthreads();
    const double M = (double)ns.M, invS = ns.S > 0.0 ? 1.0 / ns.S : 0.0;
    const int ft = first_tok;
    const size_t off = ((size_t)b * T + node) * V;
    const int s0 = split * kSegElems;
    float x[kElemsPerThread], q[kElemsPerThread];
    load_segment<VEC>(logits + off, s0, V, x);
    load_segment<VEC>(dprobs + off, s0, V, q);
    double z = 0.0, qs = 0.0;
#pragma unroll
    for (int k = 0; k < kElemsPerThread; ++k) {
        const int e = elem_index<VEC>(s0, k);
        if (e < V) {
            const double p = exp(((double)x[k] - M) * inv_tau) * invS;
            const double qd = (double)q[k];
            const double r = p - qd;
            z += r > 0.0 ? r : 0.0;
            qs += (e == ft) ? 0.0 : qd;
        }
    }
    z = block_sum(z, scratch);
    qs = block_sum(qs, scratch);
    if (threadIdx.x == 0) {
        ResPartial r;
        r.Z = z, r.Q = qs;
        resp[((size_t)b * T + node) * splits + split] = r;
    }
}

// ----------------------------------------------------------------------------- kernel 3
struct WalkShared {
    int32_t par[S4C_MAX_T];
    int32_t tok[S4C_MAX_T];
    float uni[S4C_MAX_T];
    int depth[S4C_MAX_T];
    uint32_t anc[S4C_MAX_T][S4C_MASK_WORDS];
    double nS[S4C_MAX_T];
    double nZ[S4C_MAX_T];
    double nQ[S4C_MAX_T];
    float nM[S4C_MAX_T];
    int nArg[S4C_MAX_T];
    // rejection chain at the current node
    int cx[S4C_MAX_T];
    double cinvZ[S4C_MAX_T];  // 1/Z_j, or 0 when Z_j == 0 (p kept)
    double cinvs[S4C_MAX_T];  // 1/s_j
    double scratch[33];
    double wsum[kWalkThreads / 32];
    int wlast[kWalkThreads / 32];
    int flag;
    int result_tok;
};

// p and q of vocabulary entry v after r rejections at the current node.
__device__ __forceinline__ void chain_eval(double p0, double q0, int v, int r, const WalkShared& sh, double& p,
                                           double& q) {
    p = p0, q = q0;
    for (int j = 0; j < r; ++j) {
        double res = p - q;
        res = res > 0.0 ? res : 0.0;
        const double pn = sh.cinvZ[j] > 0.0 ? res * sh.cinvZ[j] : p;
        if (v == sh.cx[j]) q = 0.0;
        q *= sh.cinvs[j];
        p = pn;
    }
}

template <bool STOCH>
__global__ void __launch_bounds__(kWalkThreads)
accept_walk_kernel(const float* __restrict__ logits, const float* __restrict__ dprobs,
                   const int32_t* __restrict__ tokens, const int32_t* __restrict__ parent,
                   const int32_t* __restrict__ n_nodes, const float* __restrict__ uniforms, int T, int V,
                   int max_depth, double inv_tau, int splits, const RowPartial* __restrict__ rowp,
                   const ResPartial* __restrict__ resp, const NodeStats* __restrict__ nodes,
                   int32_t* __restrict__ accept_len, int32_t* __restrict__ path, int32_t* __restrict__ next_token,
                   uint8_t* __restrict__ near_tie, int32_t* __restrict__ status) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    WalkShared& sh = *reinterpret_cast<WalkShared*>(smem_raw);
    const int b = blockIdx.x, tid = threadIdx.x;
    const int n = n_nodes ? n_nodes[b] : T;
    int32_t* pth = path + (size_t)b * (max_depth + 1);

    for (int i = tid; i < T; i += blockDim.x) {
        sh.par[i] = parent[(size_t)b * T + i];
        sh.tok[i] = tokens[(size_t)b * T + i];
        sh.uni[i] = (STOCH && uniforms) ? uniforms[(size_t)b * T + i] : 0.f;
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
    if (tid == 0 && status) status[b] = flags;
    if (flags) {
        for (int j = tid; j <= max_depth; j += blockDim.x) pth[j] = -1;
        if (tid == 0) accept_len[b] = -1, next_token[b] = -1;
        return;
    }

    // per-node statistics
    for (int i = tid; i < n; i += blockDim.x) {
        if (STOCH) {
            const NodeStats ns = nodes[(size_t)b * T + i];
            double z = 0.0, q = 0.0;
            const ResPartial* rp = resp + ((size_t)b * T + i) * splits;
            for (int s = 0; s < splits; ++s) z += rp[s].Z, q += rp[s].Q;
            sh.nS[i] = ns.S, sh.nM[i] = ns.M, sh.nArg[i] = ns.idx, sh.nZ[i] = z, sh.nQ[i] = q;
        } else {
            const NodeStats ns = merge_row(rowp + ((size_t)b * T + i) * splits, splits, inv_tau, false);
            sh.nArg[i] = ns.idx;
        }
    }
    __syncthreads();

    if (!STOCH) {
        if (tid == 0) {
            // ok[] as a bitmask; parent[i] < i so one ascending sweep suffices
            uint32_t ok[S4C_MASK_WORDS] = {1u, 0, 0, 0};
            int e = 0;
            for (int i = 1; i < n; ++i) {
                const int p = sh.par[i];
                if (((ok[p >> 5] >> (p & 31)) & 1u) && sh.tok[i] == sh.nArg[p]) {
                    ok[i >> 5] |= 1u << (i & 31);
                    if (sh.depth[i] > sh.depth[e]) e = i;
                }
            }
            for (int j = 0; j <= max_depth; ++j) pth[j] = -1;
            for (int t = e; t >= 0; t = sh.par[t]) pth[sh.depth[t]] = t;
            accept_len[b] = sh.depth[e];
            next_token[b] = sh.nArg[e];
        }
        return;
    }

    // ---- speculative-sampling walk: every thread follows the same control flow on the same scalars
    int cur = 0;
    for (int guard = 0; guard <= T; ++guard) {
        const float* lrow = logits + ((size_t)b * T + cur) * V;
        const float* qrow = dprobs + ((size_t)b * T + cur) * V;
        const double M = (double)sh.nM[cur];
        const double invS = sh.nS[cur] > 0.0 ? 1.0 / sh.nS[cur] : 0.0;
        int r = 0, accepted = -1;
        for (int c = cur + 1; c < n; ++c) {
            if (sh.par[c] != cur) continue;
            const int x = sh.tok[c];
            double px, qx;
            chain_eval(exp(((double)__ldg(lrow + x) - M) * inv_tau) * invS, (double)__ldg(qrow + x), x, r, sh, px, qx);
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
            // rejected: residual mass and the draft mass left once x is removed
            double Z, s;
            if (r == 0) {
                Z = sh.nZ[cur], s = sh.nQ[cur];
            } else {
                double z = 0.0, qs = 0.0;
                for (int v = tid; v < V; v += blockDim.x) {
                    double pv, qv;
                    chain_eval(exp(((double)__ldg(lrow + v) - M) * inv_tau) * invS, (double)__ldg(qrow + v), v, r, sh,
                               pv, qv);
                    const double res = pv - qv;
                    z += res > 0.0 ? res : 0.0;
                    qs += (v == x) ? 0.0 : qv;
                }
                Z = block_sum(z, sh.scratch);
                s = block_sum(qs, sh.scratch);
            }
            __syncthreads();  // everyone has finished reading the chain before it grows
            if (tid == 0) {
                sh.cx[r] = x;
                sh.cinvZ[r] = Z > 0.0 ? 1.0 / Z : 0.0;
                sh.cinvs[r] = s > 0.0 ? 1.0 / s : 0.0;
            }
            __syncthreads();
            ++r;
            if (!(s > 0.0)) break;
        }
        if (accepted >= 0) {
            cur = accepted;
            __syncthreads();
            continue;
        }

        // ---- final token: inverse CDF over the current p at `cur` (Eq. 12 at a fork; plain target at a leaf)
        const int lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
        const int seg = ((V + nwarps - 1) / nwarps + 31) / 32 * 32;  // contiguous span per warp
        const int w0 = warp * seg, w1 = min(V, w0 + seg);
        double acc = 0.0;
        int last = -1;
        for (int v = w0 + lane; v < w1; v += 32) {
            double pv, qv;
            chain_eval(exp(((double)__ldg(lrow + v) - M) * inv_tau) * invS, (double)__ldg(qrow + v), v, r, sh, pv, qv);
            acc += pv;
            if (pv > 0.0) last = v;
        }
        acc = warp_sum(acc);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) last = max(last, __shfl_xor_sync(0xffffffffu, last, o));
        if (lane == 0) sh.wsum[warp] = acc, sh.wlast[warp] = last;
        __syncthreads();
        if (warp == 0) {
            double tot = 0.0;
            int lastpos = 0;
            for (int w = 0; w < nwarps; ++w) {
                tot += sh.wsum[w];
                lastpos = max(lastpos, sh.wlast[w]);
            }
            const double target = (double)sh.uni[0] * tot;
            double run = 0.0;
            int wstar = 0;
            for (; wstar < nwarps - 1; ++wstar) {
                if (run + sh.wsum[wstar] > target) break;
                run += sh.wsum[wstar];
            }
            int pick = -1;
            for (int base = wstar * seg; base < V && pick < 0; base += 32) {
                const int v = base + lane;
                double pv = 0.0, qv;
                if (v < V)
                    chain_eval(exp(((double)__ldg(lrow + v) - M) * inv_tau) * invS, (double)__ldg(qrow + v), v, r, sh,
                               pv, qv);
                double scan = pv;  // inclusive prefix within the group of 32
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const double t = __shfl_up_sync(0xffffffffu, scan, o);
                    if (lane >= o) scan += t;
                }
                const unsigned hit = __ballot_sync(0xffffffffu, v < V && run + scan > target);
                if (hit) pick = base + __ffs(hit) - 1;
                run += __shfl_sync(0xffffffffu, scan, 31);
            }
            if (lane == 0) {
                next_token[b] = pick >= 0 ? pick : lastpos;
                for (int j = 0; j <= max_depth; ++j) pth[j] = -1;
                for (int t = cur; t >= 0; t = sh.par[t]) pth[sh.depth[t]] = t;
                accept_len[b] = sh.depth[cur];
            }
        }
        return;
    }
}

}  // namespace s4c

extern "C" size_t s4c_tree_accept_workspace_bytes(int B, int T, int V) {
    if (B < 1 || T < 1 || V < 1) return 0;
    return s4c::accept_ws_layout(B, T, V, nullptr, nullptr);
}

extern "C" s4c_status s4c_tree_accept(const float* target_logits, const float* draft_probs, const int32_t* tokens,
                                      const int32_t* parent, const int32_t* n_nodes, float temperature,
                                      const float* uniforms, int B, int T, int V, int max_depth,
                                      int32_t* accept_len, int32_t* path, int32_t* next_token, uint8_t* near_tie,
                                      int32_t* status, void* workspace, size_t workspace_bytes, s4c_stream_t stream_) {
    using namespace s4c;
    if (!target_logits || !tokens || !parent || !accept_len || !path || !next_token) return S4C_ERR_NULL;
    if (!(temperature >= 0.f) || isinf(temperature)) return S4C_ERR_SHAPE;
    const bool stoch = temperature > 0.f;
    if (stoch && (!draft_probs || !uniforms)) return S4C_ERR_NULL;
    if (B < 0 || T < 1 || T > S4C_MAX_T || V < 1 || max_depth < 0 || max_depth >= S4C_MAX_T) return S4C_ERR_SHAPE;
    if (B > 65535) return S4C_ERR_SHAPE;  // grid z limit
    if (!aligned16(target_logits) || !aligned16(draft_probs)) return S4C_ERR_ALIGN;
    if (B == 0) return S4C_OK;
    const size_t need = accept_ws_layout(B, T, V, nullptr, nullptr);
    if (!workspace || workspace_bytes < need || !aligned256(workspace)) return S4C_ERR_WORKSPACE;
    AcceptWorkspace ws;
    accept_ws_layout(B, T, V, static_cast<char*>(workspace), &ws);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int splits = accept_splits(V);
    const bool vec = (V % 4) == 0;
    const double inv_tau = stoch ? 1.0 / (double)temperature : 1.0;
    dim3 grid(splits, T, B);

    const size_t walk_smem = sizeof(WalkShared);  // ~11 KB, below the 48 KB default limit

    if (stoch) {
        if (vec)
            accept_rowstats_kernel<true, true><<<grid, kRowThreads, 0, stream>>>(target_logits, n_nodes, T, V, inv_tau, ws.row);
        else
            accept_rowstats_kernel<true, false><<<grid, kRowThreads, 0, stream>>>(target_logits, n_nodes, T, V, inv_tau, ws.row);
        S4C_RETURN_IF_CUDA_ERROR();
        if (vec)
            accept_residual_kernel<true><<<grid, kRowThreads, 0, stream>>>(target_logits, draft_probs, tokens, parent, n_nodes,
                                                                          T, V, inv_tau, ws.row, ws.res, ws.node);
        else
            accept_residual_kernel<false><<<grid, kRowThreads, 0, stream>>>(target_logits, draft_probs, tokens, parent, n_nodes,
                                                                           T, V, inv_tau, ws.row, ws.res, ws.node);
        S4C_RETURN_IF_CUDA_ERROR();
        accept_walk_kernel<true><<<B, kWalkThreads, walk_smem, stream>>>(
            target_logits, draft_probs, tokens, parent, n_nodes, uniforms, T, V, max_depth, inv_tau, splits, ws.row, ws.res,
            ws.node, accept_len, path, next_token, near_tie, status);
    } else {
        if (vec)
            accept_rowstats_kernel<false, true><<<grid, kRowThreads, 0, stream>>>(target_logits, n_nodes, T, V, inv_tau, ws.row);
        else
            accept_rowstats_kernel<false, false><<<grid, kRowThreads, 0, stream>>>(target_logits, n_nodes, T, V, inv_tau, ws.row);
        S4C_RETURN_IF_CUDA_ERROR();
        accept_walk_kernel<false><<<B, 128, walk_smem, stream>>>(
            target_logits, draft_probs, tokens, parent, n_nodes, uniforms, T, V, max_depth, inv_tau, splits, ws.row, ws.res,
            ws.node, accept_len, path, next_token, near_tie, status);
    }
    S4C_RETURN_IF_CUDA_ERROR();
    return S4C_OK;
}

// ----------------------------------------------------------------------------- no-allocation variant
// Scratch for s4c_tree_accept_noalloc lives in the library image itself: S4C_NOALLOC_SCRATCH_BYTES of device
// memory on every GPU that loads the library, held until the process exits.  In host code the array's name
// is only a handle for the runtime, never a device address, so the address is looked up once per device.
static __device__ __align__(256) unsigned char g_accept_scratch[S4C_NOALLOC_SCRATCH_BYTES];

extern "C" s4c_status s4c_tree_accept_noalloc(const float* target_logits, const float* draft_probs,
                                              const int32_t* tokens, const int32_t* parent, const int32_t* n_nodes,
                                              float temperature, const float* uniforms, int B, int T, int V,
                                              int max_depth, int32_t* accept_len, int32_t* path, int32_t* next_token,
                                              uint8_t* near_tie, int32_t* status, s4c_stream_t stream) {
    if (B < 0 || T < 1 || T > S4C_MAX_T || V < 1) return S4C_ERR_SHAPE;
    if (B > 0 && s4c::accept_ws_layout(B, T, V, nullptr, nullptr) > (size_t)S4C_NOALLOC_SCRATCH_BYTES)
        return S4C_ERR_WORKSPACE;  // the problem needs more scratch than the built-in array holds
    static void* scratch_of_device[64] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return S4C_ERR_CUDA;
    if (!scratch_of_device[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_accept_scratch) != cudaSuccess || !p) return S4C_ERR_CUDA;
        scratch_of_device[dev] = p;
    }
    return s4c_tree_accept(target_logits, draft_probs, tokens, parent, n_nodes, temperature, uniforms, B, T, V,
                           max_depth, accept_len, path, next_token, near_tie, status, scratch_of_device[dev],
                           (size_t)S4C_NOALLOC_SCRATCH_BYTES, stream);
}
