// Tree-masked attention on CUDA cores (Section 3.2 tree mask; Figure 3): the float32 path and the
// generic fallback.
//
// Used for S4C_F32 inputs (fp32 FMA keeps the 1e-4 accuracy that tf32 tensor-core products would lose)
// and for bf16 shapes the tensor-core kernel does not take.  Split-KV: grid (splits, Hq, B); each warp
// owns one query row at a time and sweeps its split's cache slots with an online softmax, lanes spread
// over the head dimension; the tree's own slots are filtered by the ancestor bitmask built in shared
// memory from parent[].  Partial (max, sum, unnormalised output) per split go to the workspace and a
// second kernel merges them in split order (deterministic, no float atomics).
#include <math.h>

#include "s4c_common.cuh"
#include "tree_attention.cuh"

namespace s4c {

constexpr int kSimtThreads = 128;
constexpr int kSimtWarps = kSimtThreads / 32;
constexpr float kLog2e = 1.4426950408889634f;

template <typename T>
struct Elem;
template <>
struct Elem<float> {
    template <int N>
    static __device__ __forceinline__ void load(const float* p, float (&v)[N]) {
        if (N == 4) {
            const float4 t = __ldg(reinterpret_cast<const float4*>(p));
            v[0] = t.x, v[1] = t.y, v[2] = t.z, v[3] = t.w;
        } else {
            const float2 t = __ldg(reinterpret_cast<const float2*>(p));
            v[0] = t.x, v[1] = t.y;
        }
    }
    template <int N>
    static __device__ __forceinline__ void store(float* p, const float (&v)[N]) {
#pragma unroll
        for (int i = 0; i < N; ++i) p[i] = v[i];
    }
};
template <>
struct Elem<__nv_bfloat16> {
    template <int N>
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&v)[N]) {
        if (N == 4) {
            const uint2 t = __ldg(reinterpret_cast<const uint2*>(p));
            const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&t.x);
            const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&t.y);
            v[0] = __low2float(a), v[1] = __high2float(a), v[2] = __low2float(b), v[3] = __high2float(b);
        } else {
            const uint32_t t = __ldg(reinterpret_cast<const uint32_t*>(p));
            const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&t);
            v[0] = __low2float(a), v[1] = __high2float(a);
        }
    }
    template <int N>
    static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&v)[N]) {
#pragma unroll
        for (int i = 0; i < N; ++i) p[i] = __float2bfloat16_rn(v[i]);
    }
};

// Validates one sequence on one CTA; returns flags (0 = fine).  par_s/anc_s/flag_s are shared memory.
__device__ __forceinline__ int load_and_check_tree(const int32_t* __restrict__ parent, const int32_t* __restrict__ n_nodes,
                                                   const int32_t* __restrict__ cache_len, int b, int T, int C,
                                                   int32_t* par_s, uint32_t (*anc_s)[S4C_MASK_WORDS], int* flag_s, int& n,
                                                   int& L) {
    n = n_nodes ? n_nodes[b] : T;
    L = cache_len[b];
    for (int i = threadIdx.x; i < T; i += blockDim.x) par_s[i] = parent[(size_t)b * T + i];
    __syncthreads();
    int flags = build_ancestor_masks(par_s, n, T, anc_s, nullptr, flag_s);
    if (L < 0 || (long long)L + (n > 0 ? n : 0) > (long long)C) flags |= S4C_SEQ_CAPACITY;
    return flags;
}

template <typename T_, int D>
__global__ void __launch_bounds__(kSimtThreads)
tree_attention_simt_kernel(const T_* __restrict__ q, const T_* __restrict__ kc, const T_* __restrict__ vc,
                           const int32_t* __restrict__ cache_len, const int32_t* __restrict__ parent,
                           const int32_t* __restrict__ n_nodes, T_* __restrict__ out, int T, int Hq, int Hkv, int C,
                           float scale_log2, int32_t* __restrict__ status, float* __restrict__ ws) {
    constexpr int DPL = D / 32;  // head-dim elements per lane
    const int split = blockIdx.x, splits = gridDim.x, h = blockIdx.y, b = blockIdx.z;
    __shared__ int32_t par_s[S4C_MAX_T];
    __shared__ uint32_t anc_s[S4C_MAX_T][S4C_MASK_WORDS];
    __shared__ int flag_s;
    int n, L;
    const int flags = load_and_check_tree(parent, n_nodes, cache_len, b, T, C, par_s, anc_s, &flag_s, n, L);
    if (split == 0 && h == 0 && threadIdx.x == 0 && status) status[b] = flags;
    if (flags) return;

    const int total = L + n;
    const int chunk = (total + splits - 1) / splits;
    const int k0 = split * chunk, k1 = min(total, k0 + chunk);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int hk = h / (Hq / Hkv);
    const T_* kb = kc + ((size_t)b * Hkv + hk) * C * D + lane * DPL;
    const T_* vb = vc + ((size_t)b * Hkv + hk) * C * D + lane * DPL;

    for (int i = warp; i < T; i += kSimtWarps) {
        float acc[DPL];
#pragma unroll
        for (int c = 0; c < DPL; ++c) acc[c] = 0.f;
        float m = -INFINITY, l = 0.f;
        if (i < n) {
            float qv[DPL];
            Elem<T_>::template load<DPL>(q + (((size_t)b * Hq + h) * T + i) * D + lane * DPL, qv);
#pragma unroll
            for (int c = 0; c < DPL; ++c) qv[c] *= scale_log2;
            for (int j = k0; j < k1; ++j) {
                if (j >= L) {
                    const int t = j - L;
                    if (!((anc_s[i][t >> 5] >> (t & 31)) & 1u)) continue;
                }
                float kv[DPL];
                Elem<T_>::template load<DPL>(kb + (size_t)j * D, kv);
                float s = 0.f;
#pragma unroll
                for (int c = 0; c < DPL; ++c) s = fmaf(qv[c], kv[c], s);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                const float mn = fmaxf(m, s);
                const float corr = exp2f(m - mn);  // m = -inf on the first visible slot: corr = 0
                const float p = exp2f(s - mn);
                float vv[DPL];
                Elem<T_>::template load<DPL>(vb + (size_t)j * D, vv);
                l = l * corr + p;
#pragma unroll
                for (int c = 0; c < DPL; ++c) acc[c] = fmaf(acc[c], corr, p * vv[c]);
                m = mn;
            }
        }
        if (splits == 1) {
            const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll
            for (int c = 0; c < DPL; ++c) acc[c] *= inv;
            Elem<T_>::template store<DPL>(out + (((size_t)b * Hq + h) * T + i) * D + lane * DPL, acc);
        } else {
            float* w = ws + ((((size_t)b * Hq + h) * T + i) * splits + split) * (D + 2);
#pragma unroll
            for (int c = 0; c < DPL; ++c) w[lane * DPL + c] = acc[c];
            if (lane == 0) w[D] = m, w[D + 1] = l;
        }
    }
}

// grid (T, Hq, B), D threads: merges the split partials of one output row in split order.
template <typename T_, int D>
__global__ void __launch_bounds__(D)
tree_attention_combine_kernel(const float* __restrict__ ws, const int32_t* __restrict__ cache_len,
                              const int32_t* __restrict__ parent, const int32_t* __restrict__ n_nodes,
                              T_* __restrict__ out, int T, int Hq, int C, int splits, int out_rows) {
    const int i = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    __shared__ int32_t par_s[S4C_MAX_T];
    __shared__ uint32_t anc_s[S4C_MAX_T][S4C_MASK_WORDS];
    __shared__ int flag_s;
    int n, L;
    if (load_and_check_tree(parent, n_nodes, cache_len, b, T, C, par_s, anc_s, &flag_s, n, L)) return;
    const float* w = ws + (((size_t)b * Hq + h) * T + i) * splits * (D + 2);
    float M = -INFINITY;
    for (int s = 0; s < splits; ++s) M = fmaxf(M, w[s * (D + 2) + D]);
    float num = 0.f, den = 0.f;
    if (i < n && M > -INFINITY)
        for (int s = 0; s < splits; ++s) {
            const float f = exp2f(w[s * (D + 2) + D] - M);
            num = fmaf(f, w[s * (D + 2) + threadIdx.x], num);
            den = fmaf(f, w[s * (D + 2) + D + 1], den);
        }
    float r[1] = {den > 0.f ? num / den : 0.f};
    const size_t orow = out_rows ? ((size_t)b * T + i) * Hq + h : ((size_t)b * Hq + h) * T + i;
    Elem<T_>::template store<1>(out + orow * D + threadIdx.x, r);
}

int simt_splits(int B, int Hq, int C) {
    int s = ceil_div(4 * 148, B * Hq);  // ~4 CTAs of 4 warps per SM
    s = s < 1 ? 1 : s;
    const int cap = C / 32 > 0 ? C / 32 : 1;  // at least 32 slots per split
    return s > cap ? cap : (s > 64 ? 64 : s);
}

size_t simt_workspace_bytes(int B, int T, int Hq, int d, int C) {
    const int s = simt_splits(B, Hq, C);
    return s == 1 ? 0 : round_up((size_t)B * Hq * T * s * (d + 2) * sizeof(float), 256);
}

template <typename T_, int D>
static s4c_status launch_combine(const void* ws, const int32_t* cache_len, const int32_t* parent, const int32_t* n_nodes,
                                 void* out, int B, int T, int Hq, int C, int splits, cudaStream_t stream, int out_rows = 0) {
    dim3 g2(T, Hq, B);
    tree_attention_combine_kernel<T_, D><<<g2, D, 0, stream>>>(static_cast<const float*>(ws), cache_len, parent, n_nodes,
                                                              static_cast<T_*>(out), T, Hq, C, splits, out_rows);
    S4C_RETURN_IF_CUDA_ERROR();
    return S4C_OK;
}

s4c_status tree_attention_combine(const void* ws, const int32_t* cache_len, const int32_t* parent, const int32_t* n_nodes,
                                  void* out, int B, int T, int Hq, int d, int C, int splits, s4c_dtype dt,
                                  cudaStream_t stream, int out_rows) {
    if (dt == S4C_F32)
        return d == 64 ? launch_combine<float, 64>(ws, cache_len, parent, n_nodes, out, B, T, Hq, C, splits, stream, out_rows)
                       : launch_combine<float, 128>(ws, cache_len, parent, n_nodes, out, B, T, Hq, C, splits, stream, out_rows);
    return d == 64 ? launch_combine<__nv_bfloat16, 64>(ws, cache_len, parent, n_nodes, out, B, T, Hq, C, splits, stream, out_rows)
                   : launch_combine<__nv_bfloat16, 128>(ws, cache_len, parent, n_nodes, out, B, T, Hq, C, splits, stream, out_rows);
}

template <typename T_, int D>
static s4c_status launch_simt(const void* q, const void* k, const void* v, const int32_t* cache_len,
                              const int32_t* parent, const int32_t* n_nodes, void* out, int B, int T, int Hq, int Hkv,
                              int C, int span, float scale, int32_t* status, void* ws, cudaStream_t stream) {
    const int splits = simt_splits(B, Hq, span);  // shaped for the live span; the kernel splits the true length
    dim3 grid(splits, Hq, B);
    tree_attention_simt_kernel<T_, D><<<grid, kSimtThreads, 0, stream>>>(
        static_cast<const T_*>(q), static_cast<const T_*>(k), static_cast<const T_*>(v), cache_len, parent, n_nodes,
        static_cast<T_*>(out), T, Hq, Hkv, C, scale * kLog2e, status, static_cast<float*>(ws));
    S4C_RETURN_IF_CUDA_ERROR();
    if (splits > 1) return launch_combine<T_, D>(ws, cache_len, parent, n_nodes, out, B, T, Hq, C, splits, stream);
    return S4C_OK;
}

s4c_status tree_attention_simt(const void* q, const void* k, const void* v, const int32_t* cache_len,
                               const int32_t* parent, const int32_t* n_nodes, void* out, int B, int T, int Hq, int Hkv,
                               int d, int C, int span, s4c_dtype dt, float scale, int32_t* status, void* ws,
                               cudaStream_t stream) {
#define S4C_SIMT(TYPE, DD) \
    launch_simt<TYPE, DD>(q, k, v, cache_len, parent, n_nodes, out, B, T, Hq, Hkv, C, span, scale, status, ws, stream)
    if (dt == S4C_F32) {
        if (d == 64) return S4C_SIMT(float, 64);
        if (d == 128) return S4C_SIMT(float, 128);
    } else {
        if (d == 64) return S4C_SIMT(__nv_bfloat16, 64);
        if (d == 128) return S4C_SIMT(__nv_bfloat16, 128);
    }
#undef S4C_SIMT
    return S4C_ERR_UNSUPPORTED;
}

}  // namespace s4c
