// s4c_tree_build: the continuous verification tree (Section 3.2; Figure 3, left) built on the device.
//
// The shape of the tree depends on the branching factors and the node budget T only: drafts are generated vertically
// first (a chain of top-1 choices), then the tree is extended horizontally, depth by depth, with the top-k alternatives
// at every position, and growth stops at T nodes.  That is integer work on at most 128 nodes: the host lays the shape
// out once per call (breadth-first numbering: parent[i] < i, siblings contiguous and in rank order) and hands it to the
// kernels as a launch parameter.  What depends on the data is which tokens the children carry: child j of node n takes
// the j-th most probable token of draft row n.  That is a top-k selection over the vocabulary per expanded node -- a
// streaming pass over the draft probabilities, bound by HBM bandwidth (every row of an expanded node is read once):
//   tree_topk_segments_kernel  grid (vocabulary segments of 4096, expanded nodes, B): the segment sits in registers;
//                              k rounds of a warp-wide (maximum, lowest index) reduction, each round restricted to
//                              entries that rank strictly after the previous winner, give each warp's k best, and one
//                              warp selects the segment's k best among those the same way
//   tree_emit_kernel           grid (B): one warp per expanded node merges the segments' candidates the same way and
//                              writes the children's tokens; the CTA also writes parent[], position ids and n_nodes
// Ranking is (probability descending, token index ascending): ties go to the lower index, every run gives the same tree.
// No tensor cores: there is no contraction here.
#include <limits.h>
#include <math.h>

#include "s4c_common.cuh"

namespace s4c {

constexpr int kTbThreads = 256;
constexpr int kTbElems = 16;
constexpr int kTbSeg = kTbThreads * kTbElems;  // 4096 probabilities per CTA
constexpr int kMaxBranch = 16;                 // most children a node may get

struct TreeShape {  // breadth-first numbering; filled on the host
    int n;                          // nodes in use (<= T)
    int n_expanded;                 // nodes with at least one child
    int16_t parent[S4C_MAX_T];
    uint8_t depth[S4C_MAX_T];
    uint8_t first_child[S4C_MAX_T];  // index of the first child (children are contiguous); 0 = none
    uint8_t n_child[S4C_MAX_T];
    uint8_t expanded[S4C_MAX_T];     // the nodes with children, ascending
};

struct Cand {  // one candidate: probability and token
    float p;
    int tok;
};

// true iff (p, tok) ranks strictly after (pp, pt) in the order (probability descending, token ascending)
__device__ __forceinline__ bool ranks_after(float p, int tok, float pp, int pt) { return p < pp || (p == pp && tok > pt); }
// true iff (p, tok) ranks before (bp, bt)
__device__ __forceinline__ bool ranks_before(float p, int tok, float bp, int bt) { return p > bp || (p == bp && tok < bt); }

__device__ __forceinline__ void warp_best(float& p, int& tok) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float op = __shfl_xor_sync(0xffffffffu, p, o);
        const int ot = __shfl_xor_sync(0xffffffffu, tok, o);
        if (ranks_before(op, ot, p, tok)) p = op, tok = ot;
    }
}

template <bool VEC>
__global__ void __launch_bounds__(kTbThreads)
tree_topk_segments_kernel(const float* __restrict__ probs, const __grid_constant__ TreeShape shape, int T, int V,
                          int max_branch, Cand* __restrict__ cand) {
    const int seg = blockIdx.x, u = shape.expanded[blockIdx.y], b = blockIdx.z;
    const int k = shape.n_child[u];
    const float* row = probs + ((size_t)b * T + u) * V;
    const int s0 = seg * kTbSeg;
    float x[kTbElems];
    int e[kTbElems];
#pragma unroll
    for (int i = 0; i < kTbElems; ++i) e[i] = VEC ? s0 + ((i >> 2) * kTbThreads + threadIdx.x) * 4 + (i & 3) : s0 + i * kTbThreads + threadIdx.x;
    if (VEC) {
#pragma unroll
        for (int i = 0; i < kTbElems / 4; ++i) {
            float4 v = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
            if (e[4 * i] < V) v = __ldg(reinterpret_cast<const float4*>(row + e[4 * i]));  // V % 4 == 0 here
            x[4 * i + 0] = v.x, x[4 * i + 1] = v.y, x[4 * i + 2] = v.z, x[4 * i + 3] = v.w;
        }
    } else {
#pragma unroll
        for (int i = 0; i < kTbElems; ++i) x[i] = e[i] < V ? __ldg(row + e[i]) : -INFINITY;
    }
    // Every warp first selects the k best of its own 512 entries (k rounds of shuffles, no CTA barrier), leaves them in
    // shared memory, and after the one barrier warp 0 selects the segment's k best among the 8 k candidates.
    __shared__ Cand wc[kTbThreads / 32][kMaxBranch];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    {
        float pp = INFINITY;  // previous winner: nothing ranks before (+inf, -1)
        int pt = -1;
        for (int r = 0; r < k; ++r) {
            float bp = -INFINITY;
            int bt = INT_MAX;  // "no entry left": ranks after every real entry
#pragma unroll
            for (int i = 0; i < kTbElems; ++i)
                if (e[i] < V && ranks_after(x[i], e[i], pp, pt) && ranks_before(x[i], e[i], bp, bt)) bp = x[i], bt = e[i];
            warp_best(bp, bt);
            pp = bp, pt = bt;
            if (lane == 0) wc[warp][r].p = bp, wc[warp][r].tok = bt;
        }
    }
    __syncthreads();
    if (warp == 0) {
        Cand* out = cand + (((size_t)b * shape.n_expanded + blockIdx.y) * gridDim.x + seg) * max_branch;
        constexpr int NW = kTbThreads / 32;
        float pp = INFINITY;
        int pt = -1;
        for (int r = 0; r < k; ++r) {
            float bp = -INFINITY;
            int bt = INT_MAX;
            for (int s = lane; s < NW * k; s += 32) {  // candidate (warp s / k, rank s % k)
                const Cand v = wc[s / k][s % k];
                if (v.tok != INT_MAX && ranks_after(v.p, v.tok, pp, pt) && ranks_before(v.p, v.tok, bp, bt)) bp = v.p, bt = v.tok;
            }
            warp_best(bp, bt);
            pp = bp, pt = bt;
            if (lane == 0) {  // an exhausted segment (fewer than k entries) leaves (-inf, INT_MAX) in the remaining slots
                Cand c;
                c.p = bt == INT_MAX ? -INFINITY : bp, c.tok = bt;
                out[r] = c;
            }
        }
    }
}

constexpr int kEmitThreads = 256;   // 8 warps: one expanded node each at a time
constexpr int kStageCands = 512;    // candidates of one node kept in shared memory (32 segments x 16 ranks)

__global__ void __launch_bounds__(kEmitThreads)
tree_emit_kernel(const Cand* __restrict__ cand, const __grid_constant__ TreeShape shape, const int32_t* __restrict__ root_token,
                 const int32_t* __restrict__ cache_len, int T, int segs, int max_branch, int32_t* __restrict__ tokens,
                 int32_t* __restrict__ parent, int32_t* __restrict__ position, int32_t* __restrict__ n_nodes) {
    const int b = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int base = cache_len ? cache_len[b] : 0;
    for (int i = threadIdx.x; i < T; i += blockDim.x) {
        const bool used = i < shape.n;
        parent[(size_t)b * T + i] = used ? (int)shape.parent[i] : -1;
        position[(size_t)b * T + i] = used ? base + (int)shape.depth[i] : 0;
        if (i == 0) tokens[(size_t)b * T] = root_token[b];
        if (!used) tokens[(size_t)b * T + i] = 0;
    }
    if (threadIdx.x == 0) n_nodes[b] = shape.n;
    // children's tokens: one warp per expanded node, k rounds over the segments' candidates, which the warp first brings
    // into shared memory (the rounds depend on one another: from global memory each would cost a round trip)
    __shared__ Cand stage[kEmitThreads / 32][kStageCands];
    for (int w = warp; w < shape.n_expanded; w += blockDim.x >> 5) {
        const int u = shape.expanded[w], k = shape.n_child[u];
        const Cand* c = cand + ((size_t)b * shape.n_expanded + w) * segs * max_branch;
        const int total = segs * k;  // slot s: segment s / k, rank s % k
        const bool staged = total <= kStageCands;
        if (staged) {
            for (int s = lane; s < total; s += 32) stage[warp][s] = c[(size_t)(s / k) * max_branch + (s % k)];
            __syncwarp();
        }
        float pp = INFINITY;
        int pt = -1;
        for (int r = 0; r < k; ++r) {
            float bp = -INFINITY;
            int bt = INT_MAX;
            for (int s = lane; s < total; s += 32) {
                const Cand v = staged ? stage[warp][s] : c[(size_t)(s / k) * max_branch + (s % k)];
                if (v.tok != INT_MAX && ranks_after(v.p, v.tok, pp, pt) && ranks_before(v.p, v.tok, bp, bt)) bp = v.p, bt = v.tok;
            }
            warp_best(bp, bt);
            pp = bp, pt = bt;
            if (lane == 0) tokens[(size_t)b * T + shape.first_child[u] + r] = bt == INT_MAX ? 0 : bt;
        }
        __syncwarp();  // the staging row is reused for the warp's next node
    }
}

// The shape of Section 3.2, in creation order first (vertical chain, then horizontal growth depth by depth, cut at T
// nodes), then renumbered breadth-first.
static void lay_out_tree(const int32_t* branching, int D, int T, TreeShape* shape) {
    int cpar[S4C_MAX_T], cdep[S4C_MAX_T], nchild[S4C_MAX_T] = {};
    int n = 1;
    cpar[0] = -1, cdep[0] = 0;
    for (int l = 0, tip = 0; l < D && n < T; ++l) {  // vertically: the chain of top-1 choices
        cpar[n] = tip, cdep[n] = l + 1, nchild[tip] += 1;
        tip = n++;
    }
    for (int l = 1; l <= D; ++l)  // horizontally: alternatives at the same position, depth by depth
        for (int node = 0; node < n; ++node) {
            if (cdep[node] != l - 1) continue;
            while (nchild[node] < branching[l - 1] && n < T) cpar[n] = node, cdep[n] = l, nchild[node] += 1, ++n;
        }
    int order[S4C_MAX_T], newid[S4C_MAX_T];  // breadth-first visit order; children in creation order
    int head = 0, tail = 0;
    order[tail++] = 0;
    while (head < tail) {
        const int u = order[head++];
        for (int c = 0; c < n; ++c)
            if (cpar[c] == u) order[tail++] = c;
    }
    for (int i = 0; i < n; ++i) newid[order[i]] = i;
    *shape = TreeShape{};
    shape->n = n;
    for (int i = 0; i < n; ++i) {
        const int old = order[i];
        const int p = old == 0 ? -1 : newid[cpar[old]];
        shape->parent[i] = (int16_t)p;
        shape->depth[i] = (uint8_t)cdep[old];
        if (p >= 0) {
            if (shape->n_child[p] == 0) shape->first_child[p] = (uint8_t)i;
            shape->n_child[p] += 1;
        }
    }
    for (int i = 0; i < n; ++i)
        if (shape->n_child[i]) shape->expanded[shape->n_expanded++] = (uint8_t)i;
}

// The same tree from the drafter's ranked choices (topk[b, n, j] = the j-th choice after node n) instead of its
// distributions: nothing to select, the children copy their tokens.
__global__ void __launch_bounds__(128)
tree_emit_topk_kernel(const int32_t* __restrict__ topk, int k, const __grid_constant__ TreeShape shape,
                      const int32_t* __restrict__ root_token, const int32_t* __restrict__ cache_len, int T,
                      int32_t* __restrict__ tokens, int32_t* __restrict__ parent, int32_t* __restrict__ position,
                      int32_t* __restrict__ n_nodes) {
    const int b = blockIdx.x;
    const int base = cache_len ? cache_len[b] : 0;
    for (int i = threadIdx.x; i < T; i += blockDim.x) {
        const bool used = i < shape.n;
        const int p = used ? (int)shape.parent[i] : -1;
        parent[(size_t)b * T + i] = p;
        position[(size_t)b * T + i] = used ? base + (int)shape.depth[i] : 0;
        int tok = 0;
        if (i == 0)
            tok = root_token[b];
        else if (used)
            tok = topk[((size_t)b * T + p) * k + (i - (int)shape.first_child[p])];  // siblings are contiguous, in rank order
        tokens[(size_t)b * T + i] = tok;
    }
    if (threadIdx.x == 0) n_nodes[b] = shape.n;
}

static inline int tb_segments(int V) { return ceil_div(V, kTbSeg); }

}  // namespace s4c

extern "C" size_t s4c_tree_build_workspace_bytes(int B, int T, int V, int max_branch) {
    using namespace s4c;
    if (B < 1 || T < 1 || T > S4C_MAX_T || V < 1 || max_branch < 1 || max_branch > kMaxBranch) return 0;
    return round_up((size_t)B * T * tb_segments(V) * max_branch * sizeof(Cand), 256);
}

extern "C" s4c_status s4c_tree_build(const float* draft_probs, const int32_t* branching, int depth,
                                     const int32_t* root_token, const int32_t* cache_len, int B, int T, int V,
                                     int32_t* tokens, int32_t* parent, int32_t* position, int32_t* n_nodes,
                                     void* workspace, size_t workspace_bytes, s4c_stream_t stream_) {
    using namespace s4c;
    if (!draft_probs || !root_token || !tokens || !parent || !position || !n_nodes || (depth > 0 && !branching)) return S4C_ERR_NULL;
    if (B < 0 || B > 65535 || T < 1 || T > S4C_MAX_T || V < 1 || depth < 0 || depth >= S4C_MAX_T) return S4C_ERR_SHAPE;
    int max_branch = 1;
    for (int l = 0; l < depth; ++l) {
        if (branching[l] < 1 || branching[l] > kMaxBranch || branching[l] > V) return S4C_ERR_SHAPE;
        max_branch = branching[l] > max_branch ? branching[l] : max_branch;
    }
    if (!aligned16(draft_probs)) return S4C_ERR_ALIGN;
    if (B == 0) return S4C_OK;
    const size_t need = s4c_tree_build_workspace_bytes(B, T, V, max_branch);
    if (!workspace || workspace_bytes < need || !aligned256(workspace)) return S4C_ERR_WORKSPACE;
    TreeShape shape;
    lay_out_tree(branching, depth, T, &shape);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    Cand* cand = static_cast<Cand*>(workspace);
    const int segs = tb_segments(V);
    if (shape.n_expanded > 0) {
        dim3 grid(segs, shape.n_expanded, B);
        if (V % 4 == 0)
            tree_topk_segments_kernel<true><<<grid, kTbThreads, 0, stream>>>(draft_probs, shape, T, V, max_branch, cand);
        else
            tree_topk_segments_kernel<false><<<grid, kTbThreads, 0, stream>>>(draft_probs, shape, T, V, max_branch, cand);
        S4C_RETURN_IF_CUDA_ERROR();
    }
    tree_emit_kernel<<<B, kEmitThreads, 0, stream>>>(cand, shape, root_token, cache_len, T, segs, max_branch, tokens, parent, position,
                                            n_nodes);
    S4C_RETURN_IF_CUDA_ERROR();
    return S4C_OK;
}

extern "C" s4c_status s4c_tree_build_topk(const int32_t* topk, int k, const int32_t* branching, int depth,
                                          const int32_t* root_token, const int32_t* cache_len, int B, int T, int32_t* tokens,
                                          int32_t* parent, int32_t* position, int32_t* n_nodes, s4c_stream_t stream_) {
    using namespace s4c;
    if (!topk || !root_token || !tokens || !parent || !position || !n_nodes || (depth > 0 && !branching)) return S4C_ERR_NULL;
    if (B < 0 || B > 65535 || T < 1 || T > S4C_MAX_T || k < 1 || depth < 0 || depth >= S4C_MAX_T) return S4C_ERR_SHAPE;
    for (int l = 0; l < depth; ++l)
        if (branching[l] < 1 || branching[l] > k) return S4C_ERR_SHAPE;  // a node cannot have more children than ranked choices
    if (B == 0) return S4C_OK;
    TreeShape shape;
    lay_out_tree(branching, depth, T, &shape);
    tree_emit_topk_kernel<<<B, 128, 0, static_cast<cudaStream_t>(stream_)>>>(topk, k, shape, root_token, cache_len, T, tokens, parent,
                                                                            position, n_nodes);
    S4C_RETURN_IF_CUDA_ERROR();
    return S4C_OK;
}
