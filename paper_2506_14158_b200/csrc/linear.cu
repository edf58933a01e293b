// s4c_linear: the linear layers of the drafter and of a decoder layer (Eq. 3: h = Linear(concat[e, f]); Eq. 4's output
// and MLP projections) on the tcgen05 tensor cores, with what follows them fused into the epilogue -- the second input's
// columns (the concatenation never exists in memory), a bias, the gated form silu(gate) * up, a residual.
// s4c_rmsnorm and s4c_embed_gather: the layer's two small row operations (root-mean-square normalisation; Eq. 6,
// e = Embedding(t)).
//
// One CTA per (column tile of the output, row tile, share of the K range): the pipeline of the q/k/v kernel -- warp 0
// requests 64-element K slices by TMA (128-byte swizzle; slices of the first input, then of the second, against consecutive
// column ranges of the weight), warp 1 issues the products into an f32 accumulator in tensor memory, warps 2-5 read it
// (one row per thread), apply the epilogue and store 16 bytes at a time.  Gated form: a tile's accumulator holds its gate
// columns beside the same outputs' up columns (two boxes of the weight), as the q/k/v kernel keeps a rotary pair in one row.
// The launch shape -- tile width (a multiple of 16 columns), one or two 128-row accumulators per CTA, the number of CTAs
// that share a tile's K range -- is chosen per call (ln_plan); shared-out K ranges meet again in linear_finish_kernel, in
// a fixed order.  All kernels here are launched programmatically dependent.  Every wait on a barrier is bounded.
#include <cuda.h>
#include <math.h>

#include <algorithm>

#include "s4c_common.cuh"
#include "tc_primitives.cuh"

namespace s4c {

using namespace tcp;

constexpr int kLnBM = 128;       // rows per CTA (tensor-memory lanes)
constexpr int kLnBN = 256;       // most accumulator columns per CTA (the launch picks a multiple of 16: see ln_plan)
constexpr int kLnBK = 64;        // K elements per stage (one 128-byte swizzled row)
constexpr int kLnMaxStages = 12;
constexpr int kLnRingBytes = 192 * 1024;
constexpr int kLnThreads = 192;  // producer warp, issuer warp, four epilogue warps
constexpr int kLnBars = 2 * kLnMaxStages + 2;  // full[], empty[], acc_full, drain
constexpr int kLnSmemBytes = 1024 + kLnRingBytes + kLnBars * 8 + 16;

struct LnParams {
    int R, N, k1_steps, k2_steps;  // K slices of the first and of the second input
    int gate;                      // 1: the weight holds N gate rows, then N up rows; out = silu(gate) * up
    int bn, cols;                  // accumulator columns of a tile (a multiple of 16, <= 256) and the output columns they make:
                                   // cols = bn, or gated bn / 2 (the first cols accumulator columns are gate rows, the rest up rows)
    int x_rows, stages;            // rows of an input box (a multiple of 32, <= 128; 256 with two row tiles); ring stages
    int nm;                        // row tiles of 128 per CTA: 1, or 2 (two accumulators fed by one weight stream)
    const __nv_bfloat16* bias;     // [N] or null
    const __nv_bfloat16* residual; // [R, N] or null
    __nv_bfloat16* out;            // [R, N]
    float* out_f32;                // [R, N] float32 instead of `out` (the LM head's logits), or null
    int32_t* status;               // one word or null
    int splits;                    // CTAs that share a tile's K slices (grid.z); > 1: raw partial sums go to `partial`
    float* partial;                // [splits][R][N or 2N] float32, read by linear_finish_kernel
};

__device__ __forceinline__ float silu(float z) { return z / (1.f + __expf(-z)); }

__global__ void __launch_bounds__(kLnThreads, 1)
linear_kernel(const __grid_constant__ CUtensorMap map_x1, const __grid_constant__ CUtensorMap map_x2,
              const __grid_constant__ CUtensorMap map_w, const LnParams prm) {
    constexpr int SM = kLnMaxStages;
    const int S = prm.stages;
    const int bn = prm.bn;
    const int x_bytes = prm.x_rows * kLnBK * 2, stage_bytes = x_bytes + bn * kLnBK * 2;
    extern __shared__ unsigned char ln_smem_raw[];
    const uint32_t raw = smem_u32(ln_smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // swizzled tiles start on 1024-byte boundaries
    unsigned char* gen = ln_smem_raw + (base - raw);
    const uint32_t bars = base + kLnRingBytes;
    auto FULL = [&](int s) { return bars + 8u * s; };
    auto EMPTY = [&](int s) { return bars + 8u * (SM + s); };
    const uint32_t ACC_FULL = bars + 8u * (2 * SM), DRAIN = bars + 8u * (2 * SM + 1);
    volatile int* tail = reinterpret_cast<volatile int*>(gen + kLnRingBytes + kLnBars * 8);
    volatile int* tmem_slot = tail;  // written by tcgen05.alloc
    volatile int* dead = tail + 1;   // a wait was given up
    volatile int* issued_s = tail + 2;
    auto sX = [&](int s) { return base + s * stage_bytes; };
    auto sW = [&](int s) { return base + s * stage_bytes + x_bytes; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ntile = blockIdx.x, mtile = blockIdx.y;
    const int k_all = prm.k1_steps + prm.k2_steps;
    const int k_begin = (int)((long long)k_all * blockIdx.z / prm.splits), k_end = (int)((long long)k_all * (blockIdx.z + 1) / prm.splits);
    const int k_steps = k_end - k_begin;  // this CTA's share of the K slices (>= 1: the launch keeps splits <= slices)
    const int cols = prm.cols;
    const int n0 = ntile * cols;  // first output column of this tile
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) mbar_init(FULL(s), 1), mbar_init(EMPTY(s), 1);
        mbar_init(ACC_FULL, 1), mbar_init(DRAIN, 1);
        mbar_fence_init();
        *dead = 0, *issued_s = 0;
        tma_prefetch_desc(&map_x1), tma_prefetch_desc(&map_w);
        if (prm.k2_steps) tma_prefetch_desc(&map_x2);
    }
    if (warp == 1) tmem_alloc(smem_u32(const_cast<int*>(tmem_slot)), kLnBN * prm.nm);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_cta = (uint32_t)*tmem_slot;
    const uint32_t tmem = tmem_cta;
    griddep_launch_dependents();  // the kernel behind may set itself up; it waits for this one's results on its own

    if (warp == 0) {
        // ================= producer =================
        if (lane == 0) {
            // every CTA walks the K slices from a start of its own (the CTAs of a row tile read the same input tiles)
            const int k0 = (int)((blockIdx.x * 7u + blockIdx.y * 3u) % (uint32_t)k_steps);
            auto slice_of = [&](int fill) { return k_begin + (fill + k0 < k_steps ? fill + k0 : fill + k0 - k_steps); };
            auto load_w = [&](int s, int ks) {
                mbar_expect_tx(FULL(s), stage_bytes);
                tma_load_2d(sW(s), &map_w, FULL(s), ks * kLnBK, n0);
                if (prm.gate) tma_load_2d(sW(s) + cols * kLnBK * 2, &map_w, FULL(s), ks * kLnBK, prm.N + n0);  // cols gate rows, then their up rows
            };
            auto load_x = [&](int s, int ks) {
                if (ks < prm.k1_steps)
                    tma_load_2d(sX(s), &map_x1, FULL(s), ks * kLnBK, mtile * kLnBM * prm.nm);
                else
                    tma_load_2d(sX(s), &map_x2, FULL(s), (ks - prm.k1_steps) * kLnBK, mtile * kLnBM * prm.nm);
            };
            // the weights do not come from the kernel in front: the first ring of weight tiles is under way before that
            // kernel has ended; the inputs follow once it has
            const int pre = k_steps < S ? k_steps : S;
            for (int f = 0; f < pre; ++f) load_w(f, slice_of(f));
            griddep_wait();
            for (int f = 0; f < pre; ++f) load_x(f, slice_of(f));
            int fill = pre, s = pre == S ? 0 : pre;
            uint32_t ph = pre == S ? 1 : 0;
            for (; fill < k_steps; ++fill, s = s + 1 == S ? 0 : s + 1, ph ^= (s == 0)) {
                if (!mbar_wait(EMPTY(s), ph ^ 1, dead)) break;
                const int ks = slice_of(fill);
                load_w(s, ks);
                load_x(s, ks);
            }
            *issued_s = fill;
        }
        __syncwarp();
    } else if (warp == 1) {
        // ================= issuer: acc = input tile x (this tile's weight rows)^T =================
        if (lane == 0) {
            const uint32_t idesc = instr_desc_bf16(kLnBM, bn, false);
            bool ok = true;
            int s = 0;
            uint32_t ph = 0;
            griddep_wait();  // the input rows are requested only after the kernel in front has ended: the bounded waits below start then
            for (int ks = 0; ks < k_steps; ++ks, s = s + 1 == S ? 0 : s + 1, ph ^= (s == 0)) {
                ok = mbar_wait(FULL(s), ph, dead);
                if (!ok) break;
                tc_fence_after();
                const uint64_t a_desc = smem_desc_sw128(sX(s), 16, 1024), b_desc = smem_desc_sw128(sW(s), 16, 1024);
#pragma unroll
                for (int kk = 0; kk < kLnBK / 16; ++kk)  // 32 bytes per K step inside the swizzled row (field unit: 16 B)
                    tc_mma_bf16(tmem, a_desc + 2u * kk, b_desc + 2u * kk, idesc, (ks > 0 || kk > 0) ? 1u : 0u);
                if (prm.nm == 2) {  // the second 128 rows of the stage (16 KB further on) meet the same weight tile
                    const uint64_t a2_desc = smem_desc_sw128(sX(s) + kLnBM * kLnBK * 2, 16, 1024);
#pragma unroll
                    for (int kk = 0; kk < kLnBK / 16; ++kk)
                        tc_mma_bf16(tmem + kLnBN, a2_desc + 2u * kk, b_desc + 2u * kk, idesc, (ks > 0 || kk > 0) ? 1u : 0u);
                }
                tc_commit(EMPTY(s));
            }
            if (ok) tc_commit(ACC_FULL);
        }
        __syncwarp();
    } else {
        // ================= epilogue =================
        const int q = warp & 3;  // the tensor-memory lanes this warp may read: 32 q .. 32 q + 31
        griddep_wait();  // (the residual may be the result of the kernel in front, and nothing is written before that kernel has ended)
        bool ok = mbar_wait(ACC_FULL, 0, dead);
        ok = __all_sync(0xffffffffu, ok);
        if (ok) tc_fence_after();
        for (int rt = 0; ok && rt < prm.nm; ++rt) {
            const int r = (mtile * prm.nm + rt) * kLnBM + q * 32 + lane;
            const uint32_t tmem = tmem_cta + (uint32_t)(rt * kLnBN);  // this row tile's accumulator
            const bool live = r < prm.R;
            __nv_bfloat16* orow = prm.out + (size_t)(live ? r : 0) * prm.N;
            const __nv_bfloat16* rrow = prm.residual ? prm.residual + (size_t)(live ? r : 0) * prm.N : nullptr;
            if (prm.splits > 1) {
                // a share of the K slices: the raw sums go out as float32, column = weight row; linear_finish_kernel adds the
                // shares in split order and applies what follows the product
                const int w_rows = prm.gate ? 2 * prm.N : prm.N;
                float* prow = prm.partial + ((size_t)blockIdx.z * prm.R + (live ? r : 0)) * w_rows;
                for (int c = 0; c < (bn + 31) / 32; ++c) {
                    uint32_t a[32];
                    tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + c * 32, a);
                    tmem_wait_ld();
                    if (live) {
#pragma unroll
                        for (int v4 = 0; v4 < 8; ++v4) {
                            // accumulator column -> weight row: plain n0 + column; gated: the first cols are gate rows n0..,
                            // the others up rows N + n0.. (cols is a multiple of 16: four columns never straddle)
                            const int tc = c * 32 + v4 * 4;
                            const bool up_part = prm.gate && tc >= cols;
                            const int wrow = up_part ? prm.N + n0 + tc - cols : n0 + tc;
                            if (tc + 4 <= bn && wrow + 4 <= (up_part ? 2 * prm.N : prm.N))
                                *reinterpret_cast<float4*>(prow + wrow) =
                                    make_float4(__uint_as_float(a[v4 * 4]), __uint_as_float(a[v4 * 4 + 1]), __uint_as_float(a[v4 * 4 + 2]),
                                                __uint_as_float(a[v4 * 4 + 3]));
                        }
                    }
                    __syncwarp();
                }
            }
            // runs of 32 output columns; the last may be short (loads past the tile's columns stay inside the allocation)
            const int n_chunks = prm.splits > 1 ? 0 : (cols + 31) / 32;
            for (int c = 0; c < n_chunks; ++c) {
                uint32_t a[32], u[32];
                tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + c * 32, a);
                if (prm.gate) tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + cols + c * 32, u);
                tmem_wait_ld();
                if (live) {
#pragma unroll
                    for (int v8 = 0; v8 < 4; ++v8) {  // eight output columns = one 16-byte store
                        const int col = n0 + c * 32 + v8 * 8;
                        if (c * 32 + v8 * 8 + 8 > cols || col + 8 > prm.N) continue;  // (cols and N are multiples of 8)
                        float y[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            y[j] = __uint_as_float(a[v8 * 8 + j]);
                            if (prm.bias) y[j] += __bfloat162float(prm.bias[col + j]);
                        }
                        if (prm.gate) {
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                float up = __uint_as_float(u[v8 * 8 + j]);
                                if (prm.bias) up += __bfloat162float(prm.bias[prm.N + col + j]);
                                y[j] = silu(y[j]) * up;
                            }
                        }
                        if (rrow) {
                            const uint4 rv = __ldg(reinterpret_cast<const uint4*>(rrow + col));
                            const __nv_bfloat162* rp = reinterpret_cast<const __nv_bfloat162*>(&rv);
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const float2 f = __bfloat1622float2(rp[j]);
                                y[2 * j] += f.x, y[2 * j + 1] += f.y;
                            }
                        }
                        if (prm.out_f32) {  // the sums as they are (logits)
                            float4* dst = reinterpret_cast<float4*>(prm.out_f32 + (size_t)r * prm.N + col);
                            dst[0] = make_float4(y[0], y[1], y[2], y[3]), dst[1] = make_float4(y[4], y[5], y[6], y[7]);
                            continue;
                        }
                        uint32_t pk[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const __nv_bfloat162 p = __floats2bfloat162_rn(y[2 * j], y[2 * j + 1]);
                            pk[j] = *reinterpret_cast<const uint32_t*>(&p);
                        }
                        *reinterpret_cast<uint4*>(orow + col) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                }
                __syncwarp();  // the lanes took different ways; the next tensor-memory load is warp-wide
            }
        }
        if (ok) tc_fence_before();
    }
    __syncthreads();
    if (*dead) {
        // a wait was given up: nothing more is issued; what is still in flight lands before shared and tensor memory go
        if (threadIdx.x == 0) {
            const int issued = *issued_s;
            for (int s = 0; s < S; ++s) {
                int last = -1;
                for (int f = s; f < issued; f += S) last = f;
                if (last >= 0) mbar_drain(FULL(s), (last / S) & 1);
            }
        }
        if (warp == 1 && lane == 0) {
            tc_commit(DRAIN);
            mbar_drain(DRAIN, 0);
        }
        __syncthreads();
        if (threadIdx.x == 0 && prm.status) atomicOr(prm.status, S4C_SEQ_TIMEOUT);
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_cta, kLnBN * prm.nm);
    }
}

// The root-mean-square normalisation's two steps, shared by rmsnorm_kernel and by the finishing kernel that normalises the
// row it has just written, so that the fused and the separate form give the same bits: a thread's share of the sum of
// squares (explicit fused multiply-adds, columns ascending), the CTA's sum (warps in order), the scaled row.
__device__ __forceinline__ float sumsq8(float ss, const uint4& v) {
    const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float2 f = __bfloat1622float2(p[j]);
        ss = __fmaf_rn(f.y, f.y, __fmaf_rn(f.x, f.x, ss));
    }
    return ss;
}
__device__ __forceinline__ float cta_sum_256(float ss, float* red) {  // 256 threads; red: 8 floats of shared memory
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red[w];
    return tot;
}
__device__ __forceinline__ uint4 scale8(const uint4& v, const uint4& g, float scale) {
    const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
    const __nv_bfloat162* pg = reinterpret_cast<const __nv_bfloat162*>(&g);
    uint32_t pk[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float2 f = __bfloat1622float2(p[j]), w2 = __bfloat1622float2(pg[j]);
        const __nv_bfloat162 o2 = __floats2bfloat162_rn(f.x * scale * w2.x, f.y * scale * w2.y);
        pk[j] = *reinterpret_cast<const uint32_t*>(&o2);
    }
    return make_uint4(pk[0], pk[1], pk[2], pk[3]);
}

// After a product whose K slices were shared out: per output element the shares in split order, then bias, gate,
// residual, one rounding to bf16.  grid (rows), eight columns per thread at a time.  With norm_weight the CTA, which
// holds the whole row, also writes its root-mean-square normalisation (of the rounded row, as a separate call would).
__global__ void __launch_bounds__(256)
linear_finish_kernel(const float* __restrict__ partial, int splits, int R, int N, int gate, const __nv_bfloat16* __restrict__ bias,
                     const __nv_bfloat16* __restrict__ residual, __nv_bfloat16* __restrict__ out,
                     const __nv_bfloat16* __restrict__ norm_weight, float norm_eps, __nv_bfloat16* __restrict__ norm_out,
                     float* __restrict__ out_f32) {
    __shared__ float red[8];
    griddep_wait();
    griddep_launch_dependents();
    const int r = blockIdx.x;
    const int w_rows = gate ? 2 * N : N;
    float ss = 0.f;
    for (int col = threadIdx.x * 8; col < N; col += blockDim.x * 8) {
        float y[8], up[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) y[j] = 0.f, up[j] = 0.f;
        for (int z = 0; z < splits; ++z) {
            const float* p = partial + ((size_t)z * R + r) * w_rows;
            const float4 a0 = *reinterpret_cast<const float4*>(p + col), a1 = *reinterpret_cast<const float4*>(p + col + 4);
            y[0] += a0.x, y[1] += a0.y, y[2] += a0.z, y[3] += a0.w, y[4] += a1.x, y[5] += a1.y, y[6] += a1.z, y[7] += a1.w;
            if (gate) {
                const float4 u0 = *reinterpret_cast<const float4*>(p + N + col), u1 = *reinterpret_cast<const float4*>(p + N + col + 4);
                up[0] += u0.x, up[1] += u0.y, up[2] += u0.z, up[3] += u0.w, up[4] += u1.x, up[5] += u1.y, up[6] += u1.z, up[7] += u1.w;
            }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (bias) y[j] += __bfloat162float(bias[col + j]);
            if (gate) {
                if (bias) up[j] += __bfloat162float(bias[N + col + j]);
                y[j] = silu(y[j]) * up[j];
            }
            if (residual) y[j] += __bfloat162float(residual[(size_t)r * N + col + j]);
        }
        if (out_f32) {  // the sums as they are (logits); no normalisation in this form
            float4* dst = reinterpret_cast<float4*>(out_f32 + (size_t)r * N + col);
            dst[0] = make_float4(y[0], y[1], y[2], y[3]), dst[1] = make_float4(y[4], y[5], y[6], y[7]);
            continue;
        }
        uint32_t pk[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const __nv_bfloat162 p2 = __floats2bfloat162_rn(y[2 * j], y[2 * j + 1]);
            pk[j] = *reinterpret_cast<const uint32_t*>(&p2);
        }
        const uint4 packed = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        *reinterpret_cast<uint4*>(out + (size_t)r * N + col) = packed;
        ss = sumsq8(ss, packed);
    }
    if (norm_weight) {  // (uniform over the CTA)
        const float scale = rsqrtf(cta_sum_256(ss, red) / (float)N + norm_eps);
        for (int col = threadIdx.x * 8; col < N; col += blockDim.x * 8) {
            const uint4 v = *reinterpret_cast<const uint4*>(out + (size_t)r * N + col);  // this thread's own stores
            const uint4 g = __ldg(reinterpret_cast<const uint4*>(norm_weight + col));
            *reinterpret_cast<uint4*>(norm_out + (size_t)r * N + col) = scale8(v, g, scale);
        }
    }
}

// root-mean-square normalisation: one CTA per row, float32 arithmetic, one rounding to bf16
__global__ void __launch_bounds__(256)
rmsnorm_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ weight, float eps, int H,
               __nv_bfloat16* __restrict__ out) {
    __shared__ float red[8];
    const size_t row = blockIdx.x;
    const __nv_bfloat16* xr = x + row * H;
    griddep_wait();
    griddep_launch_dependents();
    float ss = 0.f;
    for (int i = threadIdx.x * 8; i < H; i += blockDim.x * 8)  // H is a multiple of 8
        ss = sumsq8(ss, __ldg(reinterpret_cast<const uint4*>(xr + i)));
    const float scale = rsqrtf(cta_sum_256(ss, red) / (float)H + eps);
    for (int i = threadIdx.x * 8; i < H; i += blockDim.x * 8) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(xr + i));
        const uint4 g = __ldg(reinterpret_cast<const uint4*>(weight + i));
        *reinterpret_cast<uint4*>(out + row * H + i) = scale8(v, g, scale);
    }
}

// Eq. 6: rows of the embedding table; a token outside the table yields a row of zeros
__global__ void __launch_bounds__(256)
embed_gather_kernel(const __nv_bfloat16* __restrict__ table, const int32_t* __restrict__ tokens, int V, int H,
                    __nv_bfloat16* __restrict__ out) {
    const size_t row = blockIdx.x;
    griddep_wait();
    griddep_launch_dependents();
    const int t = tokens[row];
    const bool ok = t >= 0 && t < V;
    for (int i = threadIdx.x * 8; i < H; i += blockDim.x * 8) {
        uint4 v = make_uint4(0, 0, 0, 0);
        if (ok) v = __ldg(reinterpret_cast<const uint4*>(table + (size_t)t * H + i));
        *reinterpret_cast<uint4*>(out + row * H + i) = v;
    }
}

// ----------------------------------------------------------------------------- host side
// A launch that may begin while the kernel in front of it on the stream is still running (programmatic dependent
// launch): every kernel of this file waits (griddepcontrol.wait) before it reads what that kernel wrote or writes anything.
template <typename... KArgs, typename... Args>
static cudaError_t ln_launch(void (*kernel)(KArgs...), dim3 grid, int threads, size_t smem, cudaStream_t stream, Args... args) {
    cudaLaunchAttribute pdl;
    pdl.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid, cfg.blockDim = dim3(threads, 1, 1), cfg.dynamicSmemBytes = smem, cfg.stream = stream;
    cfg.attrs = &pdl, cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

typedef CUresult (*LnEncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                    const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static LnEncodeTiledFn ln_encode_fn() {
    static LnEncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<LnEncodeTiledFn>(p);
    }
    return fn;
}

// [rows, H] bf16 row-major, boxes of box_rows rows x 64 elements (128 bytes), 128-byte swizzle, zero fill out of range
static bool ln_make_map(CUtensorMap* map, const void* ptr, uint64_t rows, int H, int box_rows) {
    LnEncodeTiledFn fn = ln_encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)H, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)H * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kLnBK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


// The launch shape of a product: how many output columns a CTA takes (a multiple of 16; gated: twice as many
// accumulator columns) and over how many CTAs a tile's K slices are shared out.  Every admissible pair is priced by a
// small model of this kernel on this GPU and the cheapest is launched:
//   * one CTA per SM, so CTAs run in waves of 148; a second wave of a few CTAs costs as much as a full one
//     (7B-shaped gate/up projection: 172 tiles of 64 columns took 50 us, 138 tiles of 80 take one wave);
//   * per K slice of 64 elements a CTA needs the longest of: the issuing thread's fixed ~0.3 us (four tcgen05.mma, a
//     commit, a wait -- whatever the tile's width, so narrow tiles move few bytes per issue); the tensor pipe's time for
//     128 x bn x 64 products; its share of the weight stream from HBM (what one SM pulls, ~55 GB/s, or HBM divided
//     among the CTAs of the wave; row tiles of one column tile share the weights through L2); the stage's bytes over
//     what an SM takes in from L2 (~100 GB/s); and the ring's turn-round (a slot is refilled ~1.3 us after its
//     products retire, so few deep stages starve the issuer);
//   * a shared-out K range writes and re-reads float32 partial sums and runs the finishing kernel.
// The constants are measurements of this kernel on 7B- and 8B-shaped projections (26 and 256 rows), rounded; against
// 70 measured (shape, columns, splits) points the model's choice was within 4 % of the best measured one.
struct LnPlan {
    int bn, splits, x_rows, stages, cols_per_tile, m_tiles, n_tiles, nm;
};
static LnPlan ln_plan(int R, int K1, int K2, int N, int gate) {
    constexpr double kIssueUs = 0.30, kMmaUsPerCol = 0.27 / 256.0, kSmBytesPerUs = 55e3, kHbmBytesPerUs = 6.4e6, kL2BytesPerUs = 100e3,
                     kTurnUs = 1.3, kWaveUs = 2.5, kFinishUs = 3.0, kPartialBytesPerUs = 4.0e6, kIssueTwo = 1.5;
    constexpr int kSms = 148;
    const int k_steps = (K1 + K2) / kLnBK;
    const int w_rows = gate ? 2 * N : N;
    LnPlan best = {};
    double best_us = 1e30;
    // more than 128 rows: one row tile per CTA (the row tiles of a column tile share the weights through L2), or two
    // accumulators per CTA fed by one weight stream (half the weight traffic into the SM, twice the products per slice)
    for (int nm = 1; nm <= (R > kLnBM ? 2 : 1); ++nm) {
        const int m_tiles = ceil_div(R, kLnBM * nm);
        const int x_rows = nm == 2 ? 2 * kLnBM : (R > kLnBM ? kLnBM : (int)round_up((size_t)R, 32));
        const int spare = x_rows < kLnBM ? kLnBM * kLnBK * 2 : 0;  // (a product reads 128 rows from a stage's start: see the q/k/v kernel)
        for (int cols = 16; cols <= (gate ? kLnBN / 2 : kLnBN); cols += 16) {
            const int bn = gate ? 2 * cols : cols;
            const int stage_bytes = (x_rows + bn) * kLnBK * 2;
            const int stages = std::min(kLnMaxStages, (kLnRingBytes - spare) / stage_bytes);
            if (stages < 3) continue;
            const int n_tiles = ceil_div(N, cols);
            if (cols > 16 && ceil_div(N, cols - 16) == n_tiles) continue;  // the narrower tile covers N with as many CTAs
            for (int splits = 1; splits <= 8; ++splits) {
                if (splits > 1 && k_steps / splits < 4) break;
                const int ctas = n_tiles * m_tiles * splits, k_per = ceil_div(k_steps, splits);
                double us = 0.0;
                for (int left = ctas; left > 0; left -= kSms) {
                    const int active = std::min(left, kSms);
                    const double mma = kMmaUsPerCol * bn * nm;
                    const double hbm = bn * (kLnBK * 2.0) / m_tiles / std::min(kSmBytesPerUs, kHbmBytesPerUs / active);
                    const double slice = std::max(std::max(std::max(kIssueUs * (nm == 2 ? kIssueTwo : 1.0), mma),
                                                           std::max(hbm, stage_bytes / kL2BytesPerUs)),
                                                  (kTurnUs + mma) / stages);
                    us += kWaveUs + k_per * slice;
                }
                if (splits > 1) us += kFinishUs + 2.0 * splits * R * (double)w_rows * sizeof(float) / kPartialBytesPerUs;
                if (us < best_us) {
                    best_us = us;
                    best.bn = bn, best.splits = splits, best.x_rows = x_rows, best.stages = stages, best.cols_per_tile = cols;
                    best.m_tiles = m_tiles, best.n_tiles = n_tiles, best.nm = nm;
                }
            }
        }
    }
    return best;
}

}  // namespace s4c

extern "C" size_t s4c_linear_workspace_bytes(int R, int K1, int K2, int N, int gate) {
    using namespace s4c;
    if (R < 1 || N < 8 || K1 < kLnBK || K2 < 0) return 0;
    const LnPlan p = ln_plan(R, K1, K2, N, gate);
    return p.splits > 1 ? round_up((size_t)p.splits * R * (gate ? 2 * N : N) * sizeof(float), 256) : 0;
}

namespace s4c {
// s4c_linear, and s4c_linear_rmsnorm when norm_weight is given (norm_out = rmsnorm(out))
static s4c_status ln_run(const void* x1, const void* x2, const void* w, const void* bias, const void* residual, void* out, int R,
                         int K1, int K2, int N, int gate, const void* norm_weight, float norm_eps, void* norm_out, int32_t* status,
                         void* workspace, size_t workspace_bytes, s4c_stream_t stream_, bool out_is_f32 = false) {
    if (!x1 || !w || !out || (K2 > 0 && !x2) || (norm_weight && !norm_out)) return S4C_ERR_NULL;
    if (R < 0 || N < 8 || N % 8 != 0 || K1 < kLnBK || K1 % kLnBK != 0 || K2 < 0 || K2 % kLnBK != 0) return S4C_ERR_SHAPE;
    if (norm_weight && !(norm_eps >= 0.f)) return S4C_ERR_SHAPE;
    if (!aligned16(x1) || !aligned16(w) || !aligned16(out) || (x2 && !aligned16(x2)) || (residual && !aligned16(residual)) ||
        (norm_weight && (!aligned16(norm_weight) || !aligned16(norm_out))))
        return S4C_ERR_ALIGN;
    if (R == 0) return S4C_OK;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const LnPlan pl = ln_plan(R, K1, K2, N, gate);
    const size_t need = pl.splits > 1 ? round_up((size_t)pl.splits * R * (gate ? 2 * N : N) * sizeof(float), 256) : 0;
    if (need && (!workspace || workspace_bytes < need || !aligned256(workspace))) return S4C_ERR_WORKSPACE;
    if (status && cudaMemsetAsync(status, 0, sizeof(int32_t), stream) != cudaSuccess) {
        cudaGetLastError();
        return S4C_ERR_CUDA;
    }
    const int w_rows = gate ? 2 * N : N;
    CUtensorMap map_x1, map_x2, map_w;
    if (!ln_make_map(&map_x1, x1, (uint64_t)R, K1, pl.x_rows) ||
        !ln_make_map(&map_x2, K2 > 0 ? x2 : x1, (uint64_t)R, K2 > 0 ? K2 : K1, pl.x_rows) ||
        !ln_make_map(&map_w, w, (uint64_t)w_rows, K1 + K2, pl.cols_per_tile))
        return S4C_ERR_CUDA;
    static bool configured[64] = {};  // the dynamic shared memory opt-in is per device
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return S4C_ERR_CUDA;
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(linear_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kLnSmemBytes) != cudaSuccess) {
            cudaGetLastError();
            return S4C_ERR_CUDA;
        }
        configured[dev] = true;
    }
    LnParams prm;
    prm.R = R, prm.N = N, prm.k1_steps = K1 / kLnBK, prm.k2_steps = K2 / kLnBK, prm.gate = gate ? 1 : 0;
    prm.x_rows = pl.x_rows, prm.stages = pl.stages, prm.bn = pl.bn, prm.cols = pl.cols_per_tile, prm.nm = pl.nm;
    prm.bias = static_cast<const __nv_bfloat16*>(bias), prm.residual = static_cast<const __nv_bfloat16*>(residual);
    prm.out = out_is_f32 ? nullptr : static_cast<__nv_bfloat16*>(out), prm.out_f32 = out_is_f32 ? static_cast<float*>(out) : nullptr;
    prm.status = status;
    prm.splits = pl.splits, prm.partial = static_cast<float*>(workspace);
    const __nv_bfloat16* nw = static_cast<const __nv_bfloat16*>(norm_weight);
    __nv_bfloat16* no = static_cast<__nv_bfloat16*>(norm_out);
    bool ok = ln_launch(linear_kernel, dim3(pl.n_tiles, pl.m_tiles, pl.splits), kLnThreads, kLnSmemBytes, stream, map_x1, map_x2, map_w,
                        prm) == cudaSuccess;
    if (ok && pl.splits > 1)  // the finishing kernel holds whole rows: it normalises them as well
        ok = ln_launch(linear_finish_kernel, dim3(R, 1, 1), 256, 0, stream, (const float*)prm.partial, pl.splits, R, N, gate ? 1 : 0,
                       prm.bias, prm.residual, prm.out, nw, norm_eps, no, prm.out_f32) == cudaSuccess;
    else if (ok && nw)
        ok = ln_launch(rmsnorm_kernel, dim3(R, 1, 1), 256, 0, stream, (const __nv_bfloat16*)prm.out, nw, norm_eps, N, no) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        return S4C_ERR_CUDA;
    }
    return S4C_OK;
}
}  // namespace s4c

extern "C" s4c_status s4c_linear(const void* x1, const void* x2, const void* w, const void* bias, const void* residual,
                                 void* out, int R, int K1, int K2, int N, int gate, int32_t* status, void* workspace,
                                 size_t workspace_bytes, s4c_stream_t stream) {
    return s4c::ln_run(x1, x2, w, bias, residual, out, R, K1, K2, N, gate, nullptr, 0.f, nullptr, status, workspace, workspace_bytes,
                       stream);
}

extern "C" s4c_status s4c_linear_rmsnorm(const void* x1, const void* x2, const void* w, const void* bias, const void* residual,
                                         void* out, int R, int K1, int K2, int N, const void* norm_weight, float eps, void* norm_out,
                                         int32_t* status, void* workspace, size_t workspace_bytes, s4c_stream_t stream) {
    if (!norm_weight) return S4C_ERR_NULL;
    return s4c::ln_run(x1, x2, w, bias, residual, out, R, K1, K2, N, 0, norm_weight, eps, norm_out, status, workspace, workspace_bytes,
                       stream);
}

extern "C" size_t s4c_lm_head_logits_workspace_bytes(int R, int V, int H) { return s4c_linear_workspace_bytes(R, H, 0, V, 0); }

extern "C" s4c_status s4c_lm_head_logits(const void* hidden, const void* weight, int R, int V, int H, float* logits, int32_t* status,
                                         void* workspace, size_t workspace_bytes, s4c_stream_t stream) {
    return s4c::ln_run(hidden, nullptr, weight, nullptr, nullptr, logits, R, H, 0, V, 0, nullptr, 0.f, nullptr, status, workspace,
                       workspace_bytes, stream, true);
}

extern "C" s4c_status s4c_rmsnorm(const void* x, const void* weight, float eps, int R, int H, void* out, s4c_stream_t stream_) {
    using namespace s4c;
    if (!x || !weight || !out) return S4C_ERR_NULL;
    if (R < 0 || H < 8 || H % 8 != 0 || !(eps >= 0.f)) return S4C_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(weight) || !aligned16(out)) return S4C_ERR_ALIGN;
    if (R == 0) return S4C_OK;
    if (ln_launch(rmsnorm_kernel, dim3(R, 1, 1), 256, 0, static_cast<cudaStream_t>(stream_), static_cast<const __nv_bfloat16*>(x),
                  static_cast<const __nv_bfloat16*>(weight), eps, H, static_cast<__nv_bfloat16*>(out)) != cudaSuccess) {
        cudaGetLastError();
        return S4C_ERR_CUDA;
    }
    return S4C_OK;
}

extern "C" s4c_status s4c_embed_gather(const void* table, const int32_t* tokens, int R, int V, int H, void* out,
                                       s4c_stream_t stream_) {
    using namespace s4c;
    if (!table || !tokens || !out) return S4C_ERR_NULL;
    if (R < 0 || V < 1 || H < 8 || H % 8 != 0) return S4C_ERR_SHAPE;
    if (!aligned16(table) || !aligned16(out)) return S4C_ERR_ALIGN;
    if (R == 0) return S4C_OK;
    if (ln_launch(embed_gather_kernel, dim3(R, 1, 1), 256, 0, static_cast<cudaStream_t>(stream_), static_cast<const __nv_bfloat16*>(table),
                  tokens, V, H, static_cast<__nv_bfloat16*>(out)) != cudaSuccess) {
        cudaGetLastError();
        return S4C_ERR_CUDA;
    }
    return S4C_OK;
}
