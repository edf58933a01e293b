// s4c_tree_accept: acceptance of the draft tree against the target logits.
//   greedy (Section 4.1.2) and speculative sampling (Section 2; Eq. 11, Eq. 12), walked along
//   root-to-leaf paths to the longest accepted path (Section 3.2).
//
// Kernels, all HBM-streaming or latency-bound, no tensor cores (there is no contraction here):
//   per-node statistics, large problems: accept_rowstats_kernel, grid (vocab segments, T, B): every CTA holds one
//      4096-element segment of one logits row in registers (16-byte coalesced loads), reduces (max, lowest argmax)
//      with warp shuffles and, for sampling, the segment's sum of exp((x - max_seg)/tau) in float64.  The residual
//      mass after a rejection is NOT computed ahead for every node: only the few nodes on the walked path ever
//      need it, so the walk computes it when a rejection happens.
//   per-node statistics, small problems: accept_stats_cluster_kernel, one 8-CTA cluster per row with the row in
//      registers: max/argmax, sum, first-round residual mass and draft mass without the first child's token at once.
//   accept_walk_cluster_kernel  one cluster per sequence (greedy: one CTA): validates the tree, merges per-node
//      statistics, walks root to leaf.  Rejections at a node need a new residual mass; those and the final
//      inverse-CDF draw are cluster-wide passes over that single row.
// Every sum that feeds a decision is float64 with a fixed reduction order, so results do not depend on
// scheduling and agree with a sequential float64 evaluation to rounding (~1e-15 relative).
#include <float.h>
#include <math.h>

#include "s4c_common.cuh"

namespace s4c {

constexpr int kRowThreads = 256;
constexpr int kElemsPerThread = 16;
constexpr int kSegElems = kRowThreads * kElemsPerThread;  // 4096 logits per CTA

struct RowPartial {  // one vocab segment of one row
    double S;        // sum exp((x - M)/tau) over the segment (sampling only)
    float M;         // segment max
    int idx;         // lowest index attaining M
};
struct NodeStats {
    double S;
    float M;
    int idx;
};

static inline int accept_splits(int V) { return ceil_div(V, kSegElems); }

struct NodeSummary {  // per-node result of the cluster path
    double S;  // sum exp((x - M)/tau)
    double Z;  // sum max(p - q, 0)
    double Q;  // sum of q, the first child's token left out
    float M;
    int idx;   // lowest index attaining M
};

struct AcceptWorkspace {
    RowPartial* row;
    NodeSummary* summary;
};
static inline size_t accept_ws_layout(int B, int T, int V, char* base, AcceptWorkspace* ws) {
    const size_t n = (size_t)B * T * accept_splits(V);
    size_t off = 0;
    if (ws) ws->row = reinterpret_cast<RowPartial*>(base + off);
    off += round_up(n * sizeof(RowPartial), 256);
    if (ws) ws->summary = reinterpret_cast<NodeSummary*>(base + off);
    off += round_up((size_t)B * T * sizeof(NodeSummary), 256);
    return off;
}

// ----------------------------------------------------------------------------- reductions
// Maximum that keeps a NaN (fmaxf drops it): a row with a NaN logit must be reported, not silently reduced.
__device__ __forceinline__ float max_keep_nan(float a, float b) {
    float d;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}
// A row maximum the method can work with: not NaN, not +Inf (the maximum-subtracted exponent would be Inf - Inf),
// not -Inf (no token has any mass).  Single -Inf logits beside finite ones are fine: probability 0.
__device__ __forceinline__ bool usable_max(float m) { return m > -INFINITY && m < INFINITY; }

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

// exp(t) for t <= 0 in float64, about 1 ulp: t = (32 k + j) ln2/32 + r, exp(t) = 2^k * 2^(j/32) * e^r with |r| <=
// ln2/64 and a degree-6 polynomial for e^r (remainder below 4e-18).  About a third of the float64 instructions of
// the library exp, which matters because this path is otherwise bound by the float64 pipe, not by HBM.
__device__ const double kExp2Frac[32] = {
    0x1.0000000000000p+0, 0x1.059b0d3158574p+0, 0x1.0b5586cf9890fp+0, 0x1.11301d0125b51p+0,
    0x1.172b83c7d517bp+0, 0x1.1d4873168b9aap+0, 0x1.2387a6e756238p+0, 0x1.29e9df51fdee1p+0,
    0x1.306fe0a31b715p+0, 0x1.371a7373aa9cbp+0, 0x1.3dea64c123422p+0, 0x1.44e086061892dp+0,
    0x1.4bfdad5362a27p+0, 0x1.5342b569d4f82p+0, 0x1.5ab07dd485429p+0, 0x1.6247eb03a5585p+0,
    0x1.6a09e667f3bcdp+0, 0x1.71f75e8ec5f74p+0, 0x1.7a11473eb0187p+0, 0x1.82589994cce13p+0,
    0x1.8ace5422aa0dbp+0, 0x1.93737b0cdc5e5p+0, 0x1.9c49182a3f090p+0, 0x1.a5503b23e255dp+0,
    0x1.ae89f995ad3adp+0, 0x1.b7f76f2fb5e47p+0, 0x1.c199bdd85529cp+0, 0x1.cb720dcef9069p+0,
    0x1.d5818dcfba487p+0, 0x1.dfc97337b9b5fp+0, 0x1.ea4afa2a490dap+0, 0x1.f50765b6e4540p+0};

__device__ __forceinline__ double exp_nonpos(double t, const double* tab /* shared copy of kExp2Frac */) {
    if (!(t > -700.0)) return exp(t);  // result near or below the normal range (also -inf, NaN): library path
    // k = round(t * 32/ln2) by adding 1.5 * 2^52: the integer sits in the low word of the sum (no conversion or
    // rounding instruction: those run at a quarter of the float64 FMA rate)
    const double z = fma(t, 0x1.71547652b82fep+5, 6755399441055744.0);
    const int k = __double2loint(z);
    const double kd = z - 6755399441055744.0;
    double r = fma(-kd, 0x1.62e42fefa39efp-6, t);  // ln2/32, high and low part
    r = fma(-kd, 0x1.abc9e3b39803fp-61, r);
    double pl = fma(r, 1.0 / 720.0, 1.0 / 120.0);
    pl = fma(pl, r, 1.0 / 24.0);
    pl = fma(pl, r, 1.0 / 6.0);
    pl = fma(pl, r, 0.5);
    pl = fma(pl, r, 1.0);
    pl = pl * r;  // e^r - 1
    const double tj = tab[k & 31];
    const double y = fma(tj, pl, tj);  // in [1, 2.05)
    return __hiloint2double(__double2hiint(y) + ((k >> 5) << 20), __double2loint(y));  // * 2^(k >> 5), exponent stays normal
}

// exp_nonpos without the range test, for about -780 < t <= 0.  The statistics kernels raise every logit to at least
// M - 690 tau first (one float max): a term that small is below 1e-299 of the row sum either way, so neither the sum
// nor the residual mass can tell the difference, and the inner loop loses a compare and a branch per element.
__device__ __forceinline__ double exp_fast(double t, const double* tab) {
    const double z = fma(t, 0x1.71547652b82fep+5, 6755399441055744.0);
    const int k = __double2loint(z);
    const double kd = z - 6755399441055744.0;
    double r = fma(-kd, 0x1.62e42fefa39efp-6, t);
    r = fma(-kd, 0x1.abc9e3b39803fp-61, r);
    double pl = fma(r, 1.0 / 720.0, 1.0 / 120.0);
    pl = fma(pl, r, 1.0 / 24.0);
    pl = fma(pl, r, 1.0 / 6.0);
    pl = fma(pl, r, 0.5);
    pl = fma(pl, r, 1.0);
    pl = pl * r;
    const double tj = tab[k & 31];
    const double y = fma(tj, pl, tj);
    // the float floor lets t undershoot -690 by up to ulp(M)/(2 tau): the exponent is held at 2^-1000 (an integer
    // maximum, not a float64 instruction) so that it cannot wrap into the sign bit
    return __hiloint2double(__double2hiint(y) + (max(k >> 5, -1000) << 20), __double2loint(y));
}
constexpr float kExpFloorSpan = 690.f;  // in units of tau
// Rows whose float spacing at the maximum is coarser than 690 tau / 4 (a tiny temperature or enormous logits): the
// float floor M - 690 tau is no longer usable (it may round to M itself), and every logit below the maximum is at least
// ulp(M)/tau >= 172 below it in units of tau, i.e. under e^-172 of the maximum's term -- far below the rounding of the
// sum.  Such rows are summed as the number of entries equal to the maximum.
__device__ __forceinline__ bool degenerate_row(float m, float floor_span) { return floor_span < fabsf(m) * 4.8e-7f; }
__device__ __forceinline__ void fill_exp_table(double* tab) {  // every thread of the CTA; the caller synchronises
    if (threadIdx.x < 32) tab[threadIdx.x] = kExp2Frac[threadIdx.x];
}

// ----------------------------------------------------------------------------- kernel 1
template <bool VEC, bool ZERO_FILL = false>
__device__ __forceinline__ void load_segment(const float* __restrict__ row, int s0, int V, float (&x)[kElemsPerThread]) {
    const float fill = ZERO_FILL ? 0.f : -INFINITY;
    if (VEC) {
#pragma unroll
        for (int k = 0; k < kElemsPerThread / 4; ++k) {
            const int e = s0 + (k * kRowThreads + threadIdx.x) * 4;
            float4 v = make_float4(fill, fill, fill, fill);
            if (e < V) v = __ldg(reinterpret_cast<const float4*>(row + e));  // V % 4 == 0 here
            x[4 * k + 0] = v.x, x[4 * k + 1] = v.y, x[4 * k + 2] = v.z, x[4 * k + 3] = v.w;
        }
    } else {
#pragma unroll
        for (int k = 0; k < kElemsPerThread; ++k) {
            const int e = s0 + k * kRowThreads + threadIdx.x;
            x[k] = e < V ? __ldg(row + e) : fill;
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
                       double inv_tau, float floor_span, RowPartial* __restrict__ out) {
    const int split = blockIdx.x, node = blockIdx.y, b = blockIdx.z;
    if (n_nodes && node >= n_nodes[b]) return;
    const float* row = logits + ((size_t)b * T + node) * V;
    const int s0 = split * kSegElems;
    float x[kElemsPerThread];
    load_segment<VEC>(row, s0, V, x);  // -inf beyond the row

    __shared__ float sm[kRowThreads / 32];
    __shared__ int idx_s;
    __shared__ double scratch[33];
    __shared__ double tab[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (STOCH) fill_exp_table(tab);
    if (threadIdx.x == 32) idx_s = INT_MAX;

    // maximum first (one instruction per element); its lowest index is then looked up by the few threads that hold it
    // (a NaN survives this maximum, so that the segment can be reported as unusable: see below)
    float mt = x[0];
#pragma unroll
    for (int k = 1; k < kElemsPerThread; ++k) mt = max_keep_nan(mt, x[k]);
    float m = mt;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max_keep_nan(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) sm[warp] = m;
    __syncthreads();
    m = sm[0];
#pragma unroll
    for (int w = 1; w < kRowThreads / 32; ++w) m = max_keep_nan(m, sm[w]);
    const bool bad = !(m < INFINITY);  // a NaN or +Inf in the segment: the sequence will be flagged S4C_SEQ_NONFINITE
    if (!bad && mt == m) {
#pragma unroll
        for (int k = 0; k < kElemsPerThread; ++k) {  // a thread's element indices ascend with k
            const int e = elem_index<VEC>(s0, k);
            if (x[k] == m && e < V) {
                atomicMin(&idx_s, e);
                break;
            }
        }
    }

    double S = 0.0;
    if (STOCH) {
        double s = 0.0;
        if (!bad && m > -INFINITY) {
            if (degenerate_row(m, floor_span)) {
#pragma unroll
                for (int k = 0; k < kElemsPerThread; ++k) s += x[k] == m ? 1.0 : 0.0;
            } else {
                const float x_floor = m - floor_span;
                const double c = -(double)m * inv_tau;
#pragma unroll
                for (int k = 0; k < kElemsPerThread; ++k) s += exp_fast(fma((double)fmaxf(x[k], x_floor), inv_tau, c), tab);
            }
        }
        S = block_sum(s, scratch);
    } else {
        __syncthreads();  // idx_s
    }
    if (threadIdx.x == 0) {
        RowPartial r;
        r.S = S, r.M = bad ? INFINITY : m, r.idx = idx_s;  // +Inf marks the segment (and so its row) as unusable
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
    double wsum[32];  // per warp of a 1024-thread CTA
    int wlast[32];
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

// ============================================================================= cluster path
// The default path when V is a multiple of 4 and at most 8 * 1024 * 16: one thread-block cluster of 8 CTAs per
// (sequence, node) row keeps the row's logits in registers, so every logit and every draft probability is read
// from HBM exactly once and exponentiated exactly once; the row-wide maximum, sum and residual mass are merged
// across the cluster through distributed shared memory in CTA-rank order (deterministic).  The walk then runs
// as one cluster per sequence, its vocabulary-wide passes spread over the 8 CTAs.
constexpr int kCl = 8;             // CTAs per cluster
constexpr int kClEpt = 16;         // row elements per thread
constexpr int kClMaxThreads = 1024;
constexpr int kClMaxV = kCl * kClMaxThreads * kClEpt;
constexpr size_t kSegStatsMinElems = (size_t)8 << 20;  // B*T*V above which the segment kernels win (measured)

__device__ __forceinline__ uint32_t cl_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cl_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }
// Reads 8 bytes at the same shared-memory offset in CTA `rank` of the cluster.
__device__ __forceinline__ double cl_peer_f64(const double* local, uint32_t rank) {
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(local);
    uint32_t ra;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(a), "r"(rank));
    double v;
    asm volatile("ld.shared::cluster.f64 %0, [%1];" : "=d"(v) : "r"(ra));
    return v;
}

// Cluster-wide exchange area of one CTA: written by its thread 0, read by every peer after a cluster barrier.  Every
// round has fields of its own, so a round never overwrites what a slower peer may still be reading.
struct ClSlots {
    double m, idx, s, z, qs;
};

// After a cluster barrier: all 8 CTAs' values of up to two slot fields, in rank order, into shared arrays of 8.
// Call from every thread of every CTA of the cluster.
__device__ __forceinline__ void cl_gather(const double* f0, double* d0, const double* f1 = nullptr, double* d1 = nullptr) {
    cl_sync();
    if (threadIdx.x < kCl) {
        d0[threadIdx.x] = cl_peer_f64(f0, threadIdx.x);
        if (f1) d1[threadIdx.x] = cl_peer_f64(f1, threadIdx.x);
    }
    __syncthreads();
}

template <int THREADS, bool STOCH>
__global__ void __launch_bounds__(THREADS, THREADS == 1024 ? 1 : 2)
accept_stats_cluster_kernel(const float* __restrict__ logits, const float* __restrict__ dprobs,
                            const int32_t* __restrict__ tokens, const int32_t* __restrict__ parent,
                            const int32_t* __restrict__ n_nodes, int T, int V, int chunk, double inv_tau,
                            float floor_span, NodeSummary* __restrict__ out) {
    const int node = blockIdx.y, b = blockIdx.z, tid = threadIdx.x;
    const int n = n_nodes ? n_nodes[b] : T;
    if (node >= n || n > T) return;  // the whole cluster leaves together: nobody is left waiting at a barrier
    const uint32_t rank = cl_rank();
    const size_t off = ((size_t)b * T + node) * V;
    const int c0 = (int)rank * chunk;

    __shared__ ClSlots slot;
    __shared__ double gathered[kCl], gathered2[kCl];
    __shared__ double scratch[33];
    __shared__ double tab[32];
    __shared__ float wm[THREADS / 32];
    __shared__ int wi[THREADS / 32];
    __shared__ int first_tok;
    if (STOCH) fill_exp_table(tab);
    if (STOCH && tid == 32) {  // token of the first child in index order (the first one ever rejected at this node)
        int ft = -1;
        for (int c = node + 1; c < n; ++c)
            if (parent[(size_t)b * T + c] == node) {
                ft = tokens[(size_t)b * T + c];
                break;
            }
        first_tok = ft;
    }

    // ---- the row segment of this thread: 4 x 16 bytes of logits (and of draft probabilities), requested up front
    float x[kClEpt], q[kClEpt];
#pragma unroll
    for (int k = 0; k < kClEpt / 4; ++k) {
        const int e = c0 + (k * THREADS + tid) * 4;
        float4 v = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        if (e < c0 + chunk && e < V) v = __ldg(reinterpret_cast<const float4*>(logits + off + e));  // V % 4 == 0
        x[4 * k + 0] = v.x, x[4 * k + 1] = v.y, x[4 * k + 2] = v.z, x[4 * k + 3] = v.w;
    }
    if (STOCH) {
#pragma unroll
        for (int k = 0; k < kClEpt / 4; ++k) {
            const int e = c0 + (k * THREADS + tid) * 4;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (e < c0 + chunk && e < V) v = __ldg(reinterpret_cast<const float4*>(dprobs + off + e));
            q[4 * k + 0] = v.x, q[4 * k + 1] = v.y, q[4 * k + 2] = v.z, q[4 * k + 3] = v.w;
        }
    }
    auto elem = [&](int k) { return c0 + ((k >> 2) * THREADS + tid) * 4 + (k & 3); };

    auto valid = [&](int k) { return elem(k) < V && elem(k) < c0 + chunk; };

    // ---- first reduction: maximum (one instruction per element), then its lowest index from the few threads that hold it
    float mt = x[0];
#pragma unroll
    for (int k = 1; k < kClEpt; ++k) mt = max_keep_nan(mt, x[k]);
    float m = mt;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max_keep_nan(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((tid & 31) == 0) wm[tid >> 5] = m;
    if (tid == 0) wi[0] = INT_MAX;
    __syncthreads();
    m = wm[0];
    for (int w = 1; w < THREADS / 32; ++w) m = max_keep_nan(m, wm[w]);
    if (!(m < INFINITY)) m = INFINITY;  // a NaN or +Inf: the row's maximum becomes +Inf, which the walk reports
    if (mt == m) {
#pragma unroll
        for (int k = 0; k < kClEpt; ++k)  // a thread's element indices ascend with k
            if (x[k] == m && valid(k)) {
                atomicMin(&wi[0], elem(k));
                break;
            }
    }
    __syncthreads();
    if (tid == 0) slot.m = (double)m, slot.idx = (double)wi[0];  // float and int32 are exact in a double
    cl_gather(&slot.m, gathered, &slot.idx, gathered2);
    float M = -INFINITY;
    int idx = INT_MAX;
    for (int r = 0; r < kCl; ++r) argmax_combine(M, idx, (float)gathered[r], (int)gathered2[r]);
    if (!STOCH) {
        if (rank == 0 && tid == 0) {
            NodeSummary ns;
            ns.S = 0.0, ns.Z = 0.0, ns.Q = 0.0, ns.M = M, ns.idx = idx;
            out[(size_t)b * T + node] = ns;
        }
        cl_sync();  // nobody leaves while a peer may still read its slots
        return;
    }

    // ---- second reduction: e = exp((x - M)/tau), once per element, kept in registers; S = sum e
    double e[kClEpt];
    double s = 0.0;
    if (!usable_max(M)) {  // the walk flags the sequence; nothing below is used
#pragma unroll
        for (int k = 0; k < kClEpt; ++k) e[k] = 0.0;
    } else if (degenerate_row(M, floor_span)) {
#pragma unroll
        for (int k = 0; k < kClEpt; ++k) {
            e[k] = x[k] == M ? 1.0 : 0.0;
            s += e[k];
        }
    } else {
        // elements beyond the row were loaded as -inf: raised to the floor like any other far-away logit, they add
        // less than 1e-299 of the row sum
        const float x_floor = M - floor_span;
        const double c = -(double)M * inv_tau;
#pragma unroll
        for (int k = 0; k < kClEpt; ++k) {
            e[k] = exp_fast(fma((double)fmaxf(x[k], x_floor), inv_tau, c), tab);
            s += e[k];
        }
    }
    s = block_sum(s, scratch);
    if (tid == 0) slot.s = s;
    cl_gather(&slot.s, gathered);
    double S = 0.0;
    for (int r = 0; r < kCl; ++r) S += gathered[r];
    const double invS = S > 0.0 ? 1.0 / S : 0.0;

    // ---- third reduction: first-round residual mass and the draft mass without the first child's token
    const int ft = first_tok;
    double z = 0.0, qs = 0.0;
#pragma unroll
    for (int k = 0; k < kClEpt; ++k) {
        const double qd = (double)q[k];
        const double r = e[k] * invS - qd;
        z += r + fabs(r);  // 2 max(r, 0), exactly; halved below
        qs += qd;
    }
    z *= 0.5;
    // the first child's token does not count towards the draft mass that is left: one thread takes it out again
    if (tid == 0 && ft >= c0 && ft < c0 + chunk && ft < V) qs -= (double)__ldg(dprobs + off + ft);
    z = block_sum(z, scratch);
    qs = block_sum(qs, scratch);
    if (tid == 0) slot.z = z, slot.qs = qs;
    cl_gather(&slot.z, gathered, &slot.qs, gathered2);
    double Z = 0.0, Q = 0.0;
    for (int r = 0; r < kCl; ++r) Z += gathered[r], Q += gathered2[r];
    if (rank == 0 && tid == 0) {
        NodeSummary ns;
        ns.S = S, ns.Z = Z, ns.Q = Q, ns.M = M, ns.idx = idx;
        out[(size_t)b * T + node] = ns;
    }
    cl_sync();  // nobody leaves while a peer may still read its slots
}

// ---- the walk, one cluster per sequence (greedy: one CTA, no cluster, no vocabulary pass)
struct WalkClShared {
    WalkShared w;
    double tab[32];
    double slots[2][2];  // two alternating sets of (sum a, sum b): set k is rewritten two cluster barriers later
    double ga[kCl], gb[kCl];
    double tp0[S4C_MAX_T], tq0[S4C_MAX_T];  // node i's token under its parent's row: target and draft probability
    double pa[33], pb[33];                  // scratch of the paired block reduction
};

template <bool STOCH>
__global__ void __launch_bounds__(STOCH ? 1024 : 128, 1)
accept_walk_cluster_kernel(const float* __restrict__ logits, const float* __restrict__ dprobs,
                           const int32_t* __restrict__ tokens, const int32_t* __restrict__ parent,
                           const int32_t* __restrict__ n_nodes, const float* __restrict__ uniforms, int T, int V,
                           int chunk, int cache_p0, int max_depth, double inv_tau, const NodeSummary* __restrict__ nodes,
                           int seg_splits,
                           const RowPartial* __restrict__ seg_row, int32_t* __restrict__ accept_len, int32_t* __restrict__ path,
                           int32_t* __restrict__ next_token, uint8_t* __restrict__ near_tie,
                           int32_t* __restrict__ status) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    WalkClShared& cs = *reinterpret_cast<WalkClShared*>(smem_raw);
    WalkShared& sh = cs.w;
    const int b = blockIdx.y, tid = threadIdx.x;
    const uint32_t rank = STOCH ? cl_rank() : 0u;
    const bool writer = rank == 0;  // CTA 0 writes everything except the final token, which its finder writes
    const int n = n_nodes ? n_nodes[b] : T;
    int32_t* pth = path + (size_t)b * (max_depth + 1);

    for (int i = tid; i < T; i += blockDim.x) {
        sh.par[i] = parent[(size_t)b * T + i];
        sh.tok[i] = tokens[(size_t)b * T + i];
        sh.uni[i] = (STOCH && uniforms) ? uniforms[(size_t)b * T + i] : 0.f;
        if (near_tie && writer) near_tie[(size_t)b * T + i] = 0;
    }
    if (tid < 32) cs.tab[tid] = kExp2Frac[tid];
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
    if (!(flags & S4C_SEQ_BAD_PARENT)) {
        // ---- per-node statistics into shared memory (n is in 1..T here), and the check that every row is usable
        if (seg_row && STOCH) {
            // statistics came per vocabulary segment: one warp per node, lane s takes segments s, s + 32, ...; the maximum
            // and the sum go through fixed-order butterflies (the same on every run and in every CTA of the cluster)
            const int lane = tid & 31;
            for (int i = tid >> 5; i < n; i += blockDim.x >> 5) {
                const RowPartial* part = seg_row + ((size_t)b * T + i) * seg_splits;
                float M = -INFINITY;
                int idx = INT_MAX;
                for (int sg = lane; sg < seg_splits; sg += 32) argmax_combine(M, idx, part[sg].M, part[sg].idx);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    const float om = __shfl_xor_sync(0xffffffffu, M, o);
                    const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
                    argmax_combine(M, idx, om, oi);
                }
                double S = 0.0;
                if (usable_max(M))
                    for (int sg = lane; sg < seg_splits; sg += 32)
                        if (part[sg].M > -INFINITY) S += part[sg].S * exp(((double)part[sg].M - (double)M) * inv_tau);
                S = warp_sum(S);
                if (lane == 0) sh.nS[i] = S, sh.nM[i] = M, sh.nArg[i] = idx, sh.nZ[i] = 0.0, sh.nQ[i] = 0.0;
            }
        }
        for (int i = tid; i < n; i += blockDim.x) {
            if (seg_row) {
                if (!STOCH) {
                    const NodeStats ns = merge_row(seg_row + ((size_t)b * T + i) * seg_splits, seg_splits, inv_tau, false);
                    sh.nArg[i] = ns.idx, sh.nM[i] = ns.M;
                }
            } else {
                const NodeSummary ns = nodes[(size_t)b * T + i];
                sh.nS[i] = ns.S, sh.nM[i] = ns.M, sh.nArg[i] = ns.idx, sh.nZ[i] = ns.Z, sh.nQ[i] = ns.Q;
            }
        }
        __syncthreads();
        for (int i = tid; i < n; i += blockDim.x)
            if (!usable_max(sh.nM[i])) atomicOr(&sh.flag, S4C_SEQ_NONFINITE);  // a NaN or +Inf logit, or a row of -Inf only
        __syncthreads();
        flags = sh.flag;
    }
    if (tid == 0 && status && writer) status[b] = flags;
    if (flags) {  // the same in every CTA of the cluster: they all leave here, before any cluster barrier
        if (writer) {
            for (int j = tid; j <= max_depth; j += blockDim.x) pth[j] = -1;
            if (tid == 0) accept_len[b] = -1, next_token[b] = -1;
        }
        return;
    }
    if (STOCH)  // what the walk will need of the big rows, fetched by all threads at once instead of one test at a time
        for (int i = 1 + tid; i < n; i += blockDim.x) {
            const int pr = sh.par[i], x = sh.tok[i];
            const size_t at = ((size_t)b * T + pr) * V + x;
            cs.tq0[i] = (double)__ldg(dprobs + at);
            cs.tp0[i] = (double)__ldg(logits + at);  // turned into a probability below, once the parent's statistics are in
        }
    __syncthreads();
    if (STOCH)
        for (int i = 1 + tid; i < n; i += blockDim.x) {
            const int pr = sh.par[i];
            const double invS = sh.nS[pr] > 0.0 ? 1.0 / sh.nS[pr] : 0.0;
            cs.tp0[i] = exp_nonpos((cs.tp0[i] - (double)sh.nM[pr]) * inv_tau, cs.tab) * invS;
        }
    __syncthreads();
    auto write_path = [&](int end) {
        for (int j = 0; j <= max_depth; ++j) pth[j] = -1;
        for (int t = end; t >= 0; t = sh.par[t]) pth[sh.depth[t]] = t;
        accept_len[b] = sh.depth[end];
    };

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
            write_path(e);
            next_token[b] = sh.nArg[e];
        }
        return;
    }

    // ---- speculative-sampling walk: every thread of every CTA follows the same control flow on the same scalars;
    //      only the vocabulary-wide sums are split, CTA `rank` owning the elements [c0, c1)
    const int c0 = (int)rank * chunk, c1 = min(V, c0 + chunk);
    int round = 0;  // cluster-wide reductions so far (selects the slot set)
    // With room in shared memory the target probabilities of this CTA's vocabulary range at the current node are kept
    // from the first vocabulary-wide pass there to the later ones (a float64 exp per entry is most of a pass).
    double* pc = reinterpret_cast<double*>(smem_raw + ((sizeof(WalkClShared) + 15) / 16) * 16);
    // ... and, with still more room (cache_p0 == 2), the draft probabilities of the range beside them: a node where several
    // siblings are rejected takes one pass per rejection, and all but the first then run from shared memory alone
    float* qc = reinterpret_cast<float*>(pc + chunk);
    int cached_node = -1;  // node whose probabilities pc[] holds, complete after a whole pass (the same in every thread)
    // two cluster-wide sums in rank order; every thread of the cluster calls this and gets the same values
    auto cluster_sum2 = [&](double a, double bsum, double& A, double& Bs) {
        // both sums through one pair of CTA barriers, each in a fixed order
        a = warp_sum(a), bsum = warp_sum(bsum);
        if ((tid & 31) == 0) cs.pa[tid >> 5] = a, cs.pb[tid >> 5] = bsum;
        __syncthreads();
        if (tid < 32) {
            double ta = tid < (int)(blockDim.x >> 5) ? cs.pa[tid] : 0.0, tb = tid < (int)(blockDim.x >> 5) ? cs.pb[tid] : 0.0;
            ta = warp_sum(ta), tb = warp_sum(tb);
            double* set = cs.slots[round & 1];
            if (tid == 0) set[0] = ta, set[1] = tb;
        }
        double* set = cs.slots[round & 1];
        cl_sync();
        if (tid < kCl) cs.ga[tid] = cl_peer_f64(&set[0], tid), cs.gb[tid] = cl_peer_f64(&set[1], tid);
        __syncthreads();
        A = 0.0, Bs = 0.0;
        for (int r = 0; r < kCl; ++r) A += cs.ga[r], Bs += cs.gb[r];
        __syncthreads();  // ga/gb are free again
        ++round;
    };

    int cur = 0;
    for (int guard = 0; guard <= T; ++guard) {
        const float* lrow = logits + ((size_t)b * T + cur) * V;
        const float* qrow = dprobs + ((size_t)b * T + cur) * V;
        const double M = (double)sh.nM[cur];
        const double invS = sh.nS[cur] > 0.0 ? 1.0 / sh.nS[cur] : 0.0;
        auto p0_from = [&](float logit) { return exp_nonpos(((double)logit - M) * inv_tau, cs.tab) * invS; };
        // (p, q) after r rejections of up to four vocabulary entries start, start + step, ...; the loads go out
        // first (these passes are bound by the latency of the loads, not by their volume)
        auto eval4 = [&](int start, int step, int end, int rr, double (&pv)[4], double (&qv)[4]) {
            const bool hit = cache_p0 && cached_node == cur;
            float xl[4], ql[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int v = start + u * step;
                xl[u] = (v < end && !hit) ? __ldg(lrow + v) : 0.f;
                ql[u] = v < end ? ((hit && cache_p0 == 2) ? qc[v - c0] : __ldg(qrow + v)) : 0.f;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int v = start + u * step;
                pv[u] = 0.0, qv[u] = 0.0;
                if (v < end) {
                    double p0;
                    if (hit) {
                        p0 = pc[v - c0];
                    } else {
                        p0 = p0_from(xl[u]);
                        if (cache_p0) pc[v - c0] = p0;
                        if (cache_p0 == 2) qc[v - c0] = ql[u];
                    }
                    chain_eval(p0, (double)ql[u], v, rr, sh, pv[u], qv[u]);
                }
            }
        };
        int r = 0, accepted = -1;
        for (int c = cur + 1; c < n; ++c) {
            if (sh.par[c] != cur) continue;
            const int x = sh.tok[c];
            double px, qx;
            chain_eval(cs.tp0[c], cs.tq0[c], x, r, sh, px, qx);
            double ratio;
            if (qx > 0.0)
                ratio = px / qx;
            else
                ratio = px > 0.0 ? (double)INFINITY : 0.0;
            const double u = (double)sh.uni[c];
            if (tid == 0 && writer && near_tie && fabs(ratio - u) < 1e-6) near_tie[(size_t)b * T + c] = 1;
            if (u < (ratio < 1.0 ? ratio : 1.0)) {
                accepted = c;
                break;
            }
            // rejected: residual mass and the draft mass left once x is removed
            double Z, s;
            if (r == 0 && !seg_row) {  // small problems: the statistics kernel has them for every node
                Z = sh.nZ[cur], s = sh.nQ[cur];
            } else {
                double z = 0.0, qs = 0.0;
                if (!(cache_p0 && cached_node == cur))
                    // first pass at this node: the rows come from global memory in batches of four loads per thread, each
                    // batch a round trip; asking L2 for the later batches now leaves only the first at full latency
                    for (int v = c0 + tid + 4 * (int)blockDim.x; v < c1; v += blockDim.x) prefetch_l2(lrow + v), prefetch_l2(qrow + v);
                for (int v0 = c0 + tid; v0 < c1; v0 += 4 * blockDim.x) {
                    double pv[4], qv[4];
                    eval4(v0, blockDim.x, c1, r, pv, qv);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {  // entries past the end come back as (0, 0)
                        const double res = pv[u] - qv[u];
                        z += res > 0.0 ? res : 0.0;
                        qs += (v0 + u * (int)blockDim.x == x) ? 0.0 : qv[u];
                    }
                }
                cluster_sum2(z, qs, Z, s);
                cached_node = cur;  // a whole pass at this node is behind a CTA barrier: pc[] is complete
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

        // ---- final token: inverse CDF over the current p at `cur` (Eq. 12 at a fork; plain target at a leaf).
        //      Each warp sums a contiguous span of its CTA's range; the CTA totals are exchanged; the CTA whose
        //      range holds the crossing scans the one span that holds it.
        const int lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
        const int seg = ((chunk + nwarps - 1) / nwarps + 31) / 32 * 32;  // contiguous span per warp
        const int w0 = c0 + warp * seg, w1 = min(c1, w0 + seg);
        double acc = 0.0;
        int last = -1;
        if (!(cache_p0 && cached_node == cur))  // (as above: a leaf, or a fork whose residual masses came precomputed)
            for (int v = w0 + lane + 128; v < w1; v += 32) prefetch_l2(lrow + v), prefetch_l2(qrow + v);
        for (int v0 = w0 + lane; v0 < w1; v0 += 128) {
            double pv[4], qv[4];
            eval4(v0, 32, w1, r, pv, qv);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                acc += pv[u];
                if (pv[u] > 0.0) last = v0 + 32 * u;
            }
        }
        acc = warp_sum(acc);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) last = max(last, __shfl_xor_sync(0xffffffffu, last, o));
        if (lane == 0) sh.wsum[warp] = acc, sh.wlast[warp] = last;
        __syncthreads();
        cached_node = cur;  // the sums above went over the whole range: the scan below reads pc[]
        double* set = cs.slots[round & 1];
        if (tid == 0) {
            double tot = 0.0;
            int lastpos = -1;
            for (int w = 0; w < nwarps; ++w) tot += sh.wsum[w], lastpos = max(lastpos, sh.wlast[w]);
            set[0] = tot, set[1] = (double)lastpos;
        }
        cl_sync();
        if (tid < kCl) cs.ga[tid] = cl_peer_f64(&set[0], tid), cs.gb[tid] = cl_peer_f64(&set[1], tid);
        __syncthreads();
        double total = 0.0;
        int lastpos = 0;
        for (int rr = 0; rr < kCl; ++rr) total += cs.ga[rr], lastpos = max(lastpos, (int)cs.gb[rr]);
        const double target = (double)sh.uni[0] * total;
        double before = 0.0;  // mass of the ranks before the one that holds the crossing
        int rstar = -1;
        for (int rr = 0; rr < kCl; ++rr) {
            if (before + cs.ga[rr] > target) {
                rstar = rr;
                break;
            }
            before += cs.ga[rr];
        }
        if (rstar < 0) {  // the running sum never exceeds the target (u * total rounds up to the total): last token with mass
            if (writer && tid == 0) {
                next_token[b] = lastpos;
                write_path(cur);
            }
        } else if ((int)rank == rstar && warp == 0) {
            double run = before;
            int wstar = 0;
            for (; wstar < nwarps - 1; ++wstar) {
                if (run + sh.wsum[wstar] > target) break;
                run += sh.wsum[wstar];
            }
            int pick = -1;
            for (int base4 = c0 + wstar * seg; base4 < c1 && pick < 0; base4 += 128) {
                double pv4[4], qv4[4];  // four groups of 32 consecutive entries, fetched together, scanned in order
                eval4(base4 + lane, 32, c1, r, pv4, qv4);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int base = base4 + 32 * u, v = base + lane;
                    if (pick >= 0 || base >= c1) continue;  // warp-uniform
                    double scan = pv4[u];  // inclusive prefix within the group of 32
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const double t = __shfl_up_sync(0xffffffffu, scan, o);
                        if (lane >= o) scan += t;
                    }
                    const unsigned hit = __ballot_sync(0xffffffffu, v < c1 && run + scan > target);
                    if (hit) pick = base + __ffs(hit) - 1;
                    run += __shfl_sync(0xffffffffu, scan, 31);
                }
            }
            if (lane == 0) {
                // a crossing lost to the different summation order of the scan: this CTA's last token with mass
                next_token[b] = pick >= 0 ? pick : (int)cs.gb[rstar];
                write_path(cur);
            }
        }
        cl_sync();  // nobody leaves while a peer may still read its slots
        return;
    }
    cl_sync();
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

    // ---- per-node statistics: row-in-registers clusters for small problems (one launch, latency-bound), vocabulary
    //      segments of 4096 with many CTAs per SM for large ones (two launches, throughput-bound)
    const bool seg_stats = !(vec && V <= kClMaxV) || (size_t)B * T * V > kSegStatsMinElems;
    const int chunk = (int)round_up((size_t)ceil_div(V, kCl), 4);
    const float floor_span = kExpFloorSpan * (stoch ? temperature : 1.f);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kCl, attr[0].val.clusterDim.y = 1, attr[0].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.stream = stream;
    cfg.attrs = attr, cfg.numAttrs = 1;
    cudaError_t err = cudaSuccess;
    if (seg_stats) {
        if (stoch) {
            if (vec)
                accept_rowstats_kernel<true, true><<<grid, kRowThreads, 0, stream>>>(target_logits, n_nodes, T, V, inv_tau, floor_span, ws.row);
            else
                accept_rowstats_kernel<true, false><<<grid, kRowThreads, 0, stream>>>(target_logits, n_nodes, T, V, inv_tau, floor_span, ws.row);
        } else {
            if (vec)
                accept_rowstats_kernel<false, true><<<grid, kRowThreads, 0, stream>>>(target_logits, n_nodes, T, V, inv_tau, floor_span, ws.row);
            else
                accept_rowstats_kernel<false, false><<<grid, kRowThreads, 0, stream>>>(target_logits, n_nodes, T, V, inv_tau, floor_span, ws.row);
        }
        S4C_RETURN_IF_CUDA_ERROR();
    } else {
        cfg.gridDim = dim3(kCl, T, B);
#define S4C_LAUNCH_STATS(THREADS)                                                                                      \
    do {                                                                                                               \
        cfg.blockDim = dim3(THREADS, 1, 1);                                                                            \
        err = stoch ? cudaLaunchKernelEx(&cfg, accept_stats_cluster_kernel<THREADS, true>, target_logits, draft_probs, \
                                         tokens, parent, n_nodes, T, V, chunk, inv_tau, floor_span, ws.summary)                    \
                    : cudaLaunchKernelEx(&cfg, accept_stats_cluster_kernel<THREADS, false>, target_logits,            \
                                         draft_probs, tokens, parent, n_nodes, T, V, chunk, inv_tau, floor_span, ws.summary);     \
    } while (0)
        if (chunk <= 256 * kClEpt)
            S4C_LAUNCH_STATS(256);
        else if (chunk <= 512 * kClEpt)
            S4C_LAUNCH_STATS(512);
        else
            S4C_LAUNCH_STATS(1024);
#undef S4C_LAUNCH_STATS
        if (err != cudaSuccess) {
            cudaGetLastError();
            return S4C_ERR_CUDA;
        }
    }
    // ---- the walk: one cluster per sequence (greedy: one CTA, no vocabulary pass)
    const NodeSummary* summary = seg_stats ? nullptr : ws.summary;
    const RowPartial* seg_row = seg_stats ? ws.row : nullptr;
    if (stoch) {
        cfg.gridDim = dim3(kCl, B, 1);
        cfg.blockDim = dim3(1024, 1, 1);
        // room for the range's target probabilities (8 bytes per vocabulary entry of a CTA), and for its draft
        // probabilities too (4 more), next to the walk's state?
        const size_t walk_state = ((sizeof(WalkClShared) + 15) / 16) * 16;
        const size_t walk_smem_max = 227 * 1024;
        const int cache_p0 = walk_state + (size_t)chunk * 12 <= walk_smem_max ? 2 : (walk_state + (size_t)chunk * 8 <= walk_smem_max ? 1 : 0);
        cfg.dynamicSmemBytes = walk_state + (size_t)chunk * (cache_p0 == 2 ? 12 : (cache_p0 == 1 ? 8 : 0));
        {
            static bool configured[64] = {};  // the opt-in to more than 48 KB of dynamic shared memory is per device
            int dev = 0;
            if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return S4C_ERR_CUDA;
            if (!configured[dev]) {
                if (cudaFuncSetAttribute(accept_walk_cluster_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)walk_smem_max) != cudaSuccess)
                    return S4C_ERR_CUDA;
                configured[dev] = true;
            }
        }
        err = cudaLaunchKernelEx(&cfg, accept_walk_cluster_kernel<true>, target_logits, draft_probs, tokens, parent, n_nodes,
                                 uniforms, T, V, chunk, cache_p0, max_depth, inv_tau, summary, splits, seg_row,
                                 accept_len, path, next_token, near_tie, status);
        if (err != cudaSuccess) {
            cudaGetLastError();
            return S4C_ERR_CUDA;
        }
    } else {
        accept_walk_cluster_kernel<false><<<dim3(1, B), 128, sizeof(WalkClShared), stream>>>(
            target_logits, draft_probs, tokens, parent, n_nodes, uniforms, T, V, chunk, 0, max_depth, inv_tau, summary,
            splits, seg_row, accept_len, path, next_token, near_tie, status);
        S4C_RETURN_IF_CUDA_ERROR();
    }
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
    // the argument checks of s4c_tree_accept, in its order, so that both entry points name the same fault first
    if (!target_logits || !tokens || !parent || !accept_len || !path || !next_token) return S4C_ERR_NULL;
    if (!(temperature >= 0.f) || isinf(temperature)) return S4C_ERR_SHAPE;
    if (temperature > 0.f && (!draft_probs || !uniforms)) return S4C_ERR_NULL;
    if (B < 0 || B > 65535 || T < 1 || T > S4C_MAX_T || V < 1 || max_depth < 0 || max_depth >= S4C_MAX_T) return S4C_ERR_SHAPE;
    if (!s4c::aligned16(target_logits) || !s4c::aligned16(draft_probs)) return S4C_ERR_ALIGN;
    if (B == 0) return S4C_OK;
    if (s4c::accept_ws_layout(B, T, V, nullptr, nullptr) > (size_t)S4C_NOALLOC_SCRATCH_BYTES)
        return S4C_ERR_WORKSPACE;  // the problem needs more scratch than the built-in array holds
    static void* scratch_of_device[64] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return S4C_ERR_CUDA;
    }
    if (!scratch_of_device[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_accept_scratch) != cudaSuccess || !p) {
            cudaGetLastError();  // leave no error behind for the caller's next runtime call
            return S4C_ERR_CUDA;
        }
        scratch_of_device[dev] = p;
    }
    return s4c_tree_accept(target_logits, draft_probs, tokens, parent, n_nodes, temperature, uniforms, B, T, V,
                           max_depth, accept_len, path, next_token, near_tie, status, scratch_of_device[dev],
                           (size_t)S4C_NOALLOC_SCRATCH_BYTES, stream);
}
