// s4c_qkv_rope: the input side of a decoder layer in the verify pass (Section 3.2: the target's forward pass over the T
// tree tokens) -- q, k, v projections of the tree tokens' hidden states, rotary embedding of q and k at position
// committed length + depth of the node, q written in the [B,Hq,T,d] layout s4c_tree_attention reads and k, v written
// straight into the caches' tree slots (committed length + node index).  The projections never exist unrotated or in
// another layout in memory.
//
// [B*T, H] x [(Hq+2Hkv)*d, H]^T is a dense contraction: bf16 operands on the tcgen05 tensor cores, f32 accumulator in tensor
// memory.  One CTA per (head, 128-row tile): a head's d output columns are one MMA tile, so both halves of every rotary pair
// (j, j + d/2) sit in the same accumulator row.  Roles as in the LM-head kernel: warp 0 requests 64-element K slices by TMA
// (128-byte swizzle, a ring of 192 KB cut into 6 to 12 stages), warp 1 issues the products, warps 2-5 read the finished accumulator (one row per
// thread), rotate, round to bf16 and store 16 bytes at a time.  A small kernel in front checks the trees and the capacity
// and tabulates cos / sin per (node, pair) in float64; the contraction is launched programmatically dependent on it and
// only its epilogue waits for it.  Every wait on a barrier is bounded.
#include <cuda.h>
#include <math.h>

#include <algorithm>

#include "s4c_common.cuh"
#include "tc_primitives.cuh"

namespace s4c {

using namespace tcp;

constexpr int kQkBM = 128;       // rows per CTA (tensor-memory lanes)
constexpr int kQkBK = 64;        // hidden elements per stage (one 128-byte swizzled row)
constexpr int kQkMaxStages = 12;
constexpr int kQkRingBytes = 192 * 1024;  // cut into stages at launch: a stage holds the rows that exist and the head's d weight rows
constexpr int kQkThreads = 192;  // producer warp, issuer warp, four epilogue warps
constexpr int kQkBars = 2 * kQkMaxStages + 2;  // full[], empty[], acc_full, drain
constexpr int kQkSmemBytes = 1024 + kQkRingBytes + kQkBars * 8 + 16;

struct QkParams {
    int R, T, Hq, Hkv, d, C, k_steps;
    int x_rows;   // rows of a state box (a multiple of 32, <= 128): 26 rows need not move 128
    int stages;   // ring stages of x_rows + d rows of 128 bytes each
    const int32_t* row_base;   // [R]: the row's committed length, -1 = write nothing (padding node, flagged sequence)
    const float2* rope;        // [R][d/2]: (cos, sin) of the row's position times the pair's frequency
    __nv_bfloat16* q_out;      // [B,Hq,T,d]
    __nv_bfloat16* k_cache;    // [B,Hkv,C,d]
    __nv_bfloat16* v_cache;
    int32_t* status;           // [B] (may be null)
    int wait_x;                // 1: the input rows may come from the kernel directly in front (no table kernel between)
};

// Tree and capacity checks, the rows' cache bases and the rotary table.  grid (sequences, groups of kQkPrepNodes nodes):
// every CTA of a sequence checks its tree (integer work on at most 128 nodes), then tabulates its own nodes -- the float64
// power and sine / cosine are the expensive part and spread over the grid; a thread keeps one frequency.
constexpr int kQkPrepNodes = 8;
__global__ void __launch_bounds__(128)
qkv_prep_kernel(const int32_t* __restrict__ cache_len, const int32_t* __restrict__ parent, const int32_t* __restrict__ n_nodes,
                const int32_t* __restrict__ position_base, int T, int C, int d, double theta, int32_t* __restrict__ row_base,
                float2* __restrict__ rope, int32_t* __restrict__ status) {
    __shared__ int32_t par[S4C_MAX_T];
    __shared__ int depth[S4C_MAX_T];
    __shared__ uint32_t anc[S4C_MAX_T][S4C_MASK_WORDS];
    __shared__ int flag;
    griddep_launch_dependents();
    const int b = blockIdx.x, tid = threadIdx.x;
    const int t0 = blockIdx.y * kQkPrepNodes, t1 = min(T, t0 + kQkPrepNodes);
    const int n = n_nodes ? n_nodes[b] : T;
    const int L = cache_len[b];
    const int P = position_base ? position_base[b] : L;  // the root's position: the cache length unless the caller says otherwise
    for (int i = tid; i < T; i += blockDim.x) par[i] = parent[(size_t)b * T + i];
    __syncthreads();
    int flags = build_ancestor_masks(par, n, T, anc, depth, &flag);
    if (L < 0 || L + T > C || P < 0) flags |= S4C_SEQ_CAPACITY;
    if (tid == 0 && blockIdx.y == 0 && status) status[b] = flags;
    for (int t = t0 + tid; t < t1; t += blockDim.x) row_base[(size_t)b * T + t] = (!flags && t < n) ? L : -1;
    if (flags) return;
    const int half = d / 2;  // 32 or 64: divides the block size, so a thread's pair index never changes
    const int i = tid % half;
    const double freq = pow(theta, -2.0 * (double)i / (double)d);
    for (int t = t0 + tid / half; t < min(t1, n); t += blockDim.x / half) {
        double sn, cs;
        sincos((double)(P + depth[t]) * freq, &sn, &cs);
        rope[((size_t)b * T + t) * half + i] = make_float2((float)cs, (float)sn);
    }
}

__global__ void __launch_bounds__(kQkThreads, 1)
qkv_rope_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, const QkParams prm) {
    constexpr int SM = kQkMaxStages;
    const int S = prm.stages;
    const int x_bytes = prm.x_rows * kQkBK * 2, stage_bytes = x_bytes + prm.d * kQkBK * 2;
    extern __shared__ unsigned char qk_smem_raw[];
    const uint32_t raw = smem_u32(qk_smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // swizzled tiles start on 1024-byte boundaries
    unsigned char* gen = qk_smem_raw + (base - raw);
    const uint32_t bars = base + kQkRingBytes;
    auto FULL = [&](int s) { return bars + 8u * s; };
    auto EMPTY = [&](int s) { return bars + 8u * (SM + s); };
    const uint32_t ACC_FULL = bars + 8u * (2 * SM), DRAIN = bars + 8u * (2 * SM + 1);
    volatile int* tail = reinterpret_cast<volatile int*>(gen + kQkRingBytes + kQkBars * 8);
    volatile int* tmem_slot = tail;  // written by tcgen05.alloc
    volatile int* dead = tail + 1;   // a wait was given up
    volatile int* issued_s = tail + 2;
    auto sX = [&](int s) { return base + s * stage_bytes; };
    auto sW = [&](int s) { return base + s * stage_bytes + x_bytes; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int head = blockIdx.x, mtile = blockIdx.y, d = prm.d;
    const uint32_t tmem_cols = d <= 64 ? 64u : 128u;
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) mbar_init(FULL(s), 1), mbar_init(EMPTY(s), 1);
        mbar_init(ACC_FULL, 1), mbar_init(DRAIN, 1);
        mbar_fence_init();
        *dead = 0, *issued_s = 0;
        tma_prefetch_desc(&map_x), tma_prefetch_desc(&map_w);
    }
    if (warp == 1) tmem_alloc(smem_u32(const_cast<int*>(tmem_slot)), tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = (uint32_t)*tmem_slot;

    if (warp == 0) {
        // ================= producer =================
        if (lane == 0) {
            // every CTA walks the K slices from a start of its own: the CTAs of a row tile all read the same state tiles,
            // and in step they would all ask the same L2 lines at the same moment (the order of a sum's terms is free)
            const int k0 = (int)((blockIdx.x * 7u + blockIdx.y * 3u) % (uint32_t)prm.k_steps);
            auto slice_of = [&](int fill) { return fill + k0 < prm.k_steps ? fill + k0 : fill + k0 - prm.k_steps; };
            int fill = 0, s = 0;
            uint32_t ph = 0;  // the ring pass's parity (stage and parity are stepped, not divided out: S is not a constant)
            if (prm.wait_x) {
                // no table kernel in front: the weights (which no kernel of the step writes) fill the first ring while the
                // kernel that produces the input rows is still running; the rows follow once it has ended
                const int pre = prm.k_steps < S ? prm.k_steps : S;
                for (int f = 0; f < pre; ++f) {
                    mbar_expect_tx(FULL(f), stage_bytes);
                    tma_load_2d(sW(f), &map_w, FULL(f), slice_of(f) * kQkBK, head * d);
                }
                griddep_wait();
                for (int f = 0; f < pre; ++f) tma_load_2d(sX(f), &map_x, FULL(f), slice_of(f) * kQkBK, mtile * kQkBM);
                fill = pre, s = pre == S ? 0 : pre, ph = pre == S ? 1 : 0;
            }
            for (; fill < prm.k_steps; ++fill, s = s + 1 == S ? 0 : s + 1, ph ^= (s == 0)) {
                if (!mbar_wait(EMPTY(s), ph ^ 1, dead)) break;
                const int ks = slice_of(fill);
                mbar_expect_tx(FULL(s), stage_bytes);
                tma_load_2d(sX(s), &map_x, FULL(s), ks * kQkBK, mtile * kQkBM);
                tma_load_2d(sW(s), &map_w, FULL(s), ks * kQkBK, head * d);
            }
            *issued_s = fill;
        }
        __syncwarp();
    } else if (warp == 1) {
        // ================= issuer: acc = state tile x (this head's weight rows)^T =================
        if (lane == 0) {
            const uint32_t idesc = instr_desc_bf16(kQkBM, d, false);
            bool ok = true;
            int s = 0;
            uint32_t ph = 0;
            if (prm.wait_x) griddep_wait();  // the rows are requested only after the kernel in front has ended: the bounded waits start then
            for (int ks = 0; ks < prm.k_steps; ++ks, s = s + 1 == S ? 0 : s + 1, ph ^= (s == 0)) {
                ok = mbar_wait(FULL(s), ph, dead);
                if (!ok) break;
                tc_fence_after();
                const uint64_t a_desc = smem_desc_sw128(sX(s), 16, 1024), b_desc = smem_desc_sw128(sW(s), 16, 1024);
#pragma unroll
                for (int kk = 0; kk < kQkBK / 16; ++kk)  // 32 bytes per K step inside the swizzled row (field unit: 16 B)
                    tc_mma_bf16(tmem, a_desc + 2u * kk, b_desc + 2u * kk, idesc, (ks > 0 || kk > 0) ? 1u : 0u);
                tc_commit(EMPTY(s));
            }
            if (ok) tc_commit(ACC_FULL);
        }
        __syncwarp();
    } else {
        // ================= epilogue: rotate, round, store =================
        const int q = warp & 3;  // the tensor-memory lanes this warp may read: 32 q .. 32 q + 31
        const int r = mtile * kQkBM + q * 32 + lane;
        bool ok = mbar_wait(ACC_FULL, 0, dead);
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
            tc_fence_after();
            griddep_wait();  // the rows' bases and the rotary table are complete
            const int Lb = r < prm.R ? prm.row_base[r] : -1;
            const int b = r / prm.T, t = r - b * prm.T, half = d >> 1;
            __nv_bfloat16* dst = nullptr;
            bool rotate = true;
            if (Lb >= 0) {
                if (head < prm.Hq)
                    dst = prm.q_out + (((size_t)b * prm.Hq + head) * prm.T + t) * d;
                else if (head < prm.Hq + prm.Hkv)
                    dst = prm.k_cache + (((size_t)b * prm.Hkv + (head - prm.Hq)) * prm.C + Lb + t) * d;
                else
                    dst = prm.v_cache + (((size_t)b * prm.Hkv + (head - prm.Hq - prm.Hkv)) * prm.C + Lb + t) * d, rotate = false;
            }
            const float2* cs = prm.rope + (size_t)(r < prm.R ? r : 0) * half;
            for (int c = 0; c < half / 32; ++c) {  // columns [32c, 32c+32) and their partners half further on
                uint32_t lo[32], hi[32];
                tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + c * 32, lo);
                tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + half + c * 32, hi);
                tmem_wait_ld();
                if (dst) {
                    uint32_t plo[16], phi[16];
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        float a0 = __uint_as_float(lo[j]), a1 = __uint_as_float(lo[j + 1]);
                        float b0 = __uint_as_float(hi[j]), b1 = __uint_as_float(hi[j + 1]);
                        if (rotate) {
                            const float4 w = __ldg(reinterpret_cast<const float4*>(cs + c * 32 + j));  // (cos, sin) of two pairs
                            const float x0 = a0, x1 = a1;
                            a0 = x0 * w.x - b0 * w.y, b0 = b0 * w.x + x0 * w.y;
                            a1 = x1 * w.z - b1 * w.w, b1 = b1 * w.z + x1 * w.w;
                        }
                        const __nv_bfloat162 pa = __floats2bfloat162_rn(a0, a1), pb = __floats2bfloat162_rn(b0, b1);
                        plo[j >> 1] = *reinterpret_cast<const uint32_t*>(&pa), phi[j >> 1] = *reinterpret_cast<const uint32_t*>(&pb);
                    }
                    uint4* o_lo = reinterpret_cast<uint4*>(dst + c * 32);
                    uint4* o_hi = reinterpret_cast<uint4*>(dst + half + c * 32);
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        o_lo[v] = make_uint4(plo[4 * v], plo[4 * v + 1], plo[4 * v + 2], plo[4 * v + 3]);
                        o_hi[v] = make_uint4(phi[4 * v], phi[4 * v + 1], phi[4 * v + 2], phi[4 * v + 3]);
                    }
                }
            }
            tc_fence_before();
        }
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
        if (threadIdx.x == 0 && prm.status) {  // the sequences that have rows in this tile
            const int r0 = mtile * kQkBM, r1 = min(prm.R, r0 + kQkBM) - 1;
            for (int b = r0 / prm.T; b <= r1 / prm.T; ++b) atomicOr(prm.status + b, S4C_SEQ_TIMEOUT);
        }
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, tmem_cols);
    }
}

// ----------------------------------------------------------------------------- host side
typedef CUresult (*QkEncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                    const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static QkEncodeTiledFn qk_encode_fn() {
    static QkEncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<QkEncodeTiledFn>(p);
    }
    return fn;
}

// [rows, H] bf16 row-major, boxes of box_rows rows x 64 elements (128 bytes), 128-byte swizzle, zero fill out of range
static bool qk_make_map(CUtensorMap* map, const void* ptr, uint64_t rows, int H, int box_rows) {
    QkEncodeTiledFn fn = qk_encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)H, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)H * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kQkBK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static inline size_t qk_ws_layout(int B, int T, int d, char* base, int32_t** row_base, float2** rope) {
    const size_t R = (size_t)B * T;
    size_t off = 0;
    if (row_base) *row_base = reinterpret_cast<int32_t*>(base + off);
    off += round_up(R * sizeof(int32_t), 256);
    if (rope) *rope = reinterpret_cast<float2*>(base + off);
    off += round_up(R * (d / 2) * sizeof(float2), 256);
    return off;
}

}  // namespace s4c

extern "C" size_t s4c_qkv_rope_workspace_bytes(int B, int T, int d) {
    if (B < 1 || T < 1 || (d != 64 && d != 128)) return 0;
    return s4c::qk_ws_layout(B, T, d, nullptr, nullptr, nullptr);
}

namespace s4c {
// tables: the tree / rotary-table kernel runs first (s4c_qkv_rope); otherwise the tables of the call before on this
// workspace are used as they are (s4c_qkv_rope_same_tree)
static s4c_status qk_run(bool tables, const void* x, const void* w_qkv, const int32_t* cache_len, const int32_t* parent,
                         const int32_t* n_nodes, const int32_t* position_base, void* q_out, void* k_cache, void* v_cache, int B, int T, int H, int Hq, int Hkv, int d,
                         int C, float rope_theta, int32_t* status, void* workspace, size_t workspace_bytes, s4c_stream_t stream_) {
    if (!x || !w_qkv || (tables && (!cache_len || !parent)) || !q_out || !k_cache || !v_cache) return S4C_ERR_NULL;
    if (B < 0 || T < 1 || T > S4C_MAX_T || Hq < 1 || Hkv < 1 || Hq % Hkv != 0 || (d != 64 && d != 128) || C < T) return S4C_ERR_SHAPE;
    if (H < kQkBK || H % kQkBK != 0 || !(rope_theta > 1.f) || isinf(rope_theta)) return S4C_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(w_qkv) || !aligned16(q_out) || !aligned16(k_cache) || !aligned16(v_cache)) return S4C_ERR_ALIGN;
    if (B == 0) return S4C_OK;
    int32_t* row_base;
    float2* rope;
    const size_t need = qk_ws_layout(B, T, d, nullptr, nullptr, nullptr);
    if (!workspace || workspace_bytes < need || !aligned256(workspace)) return S4C_ERR_WORKSPACE;
    qk_ws_layout(B, T, d, static_cast<char*>(workspace), &row_base, &rope);
    const int R = B * T, heads = Hq + 2 * Hkv;
    CUtensorMap map_x, map_w;
    // the ring: a stage holds one K slice of the rows that exist and of the head's weight rows; as many stages as fit.  The
    // product always reads 128 rows from a stage's start: one spare tile at the ring's end keeps that read inside the ring
    // when a stage is shorter than a full tile.
    const int x_rows = R > kQkBM ? kQkBM : (int)round_up((size_t)R, 32);
    const int stage_bytes = x_rows * kQkBK * 2 + d * kQkBK * 2;
    const int stages = std::min(kQkMaxStages, (kQkRingBytes - (x_rows < kQkBM ? kQkBM * kQkBK * 2 : 0)) / stage_bytes);
    if (!qk_make_map(&map_x, x, (uint64_t)R, H, x_rows) || !qk_make_map(&map_w, w_qkv, (uint64_t)heads * d, H, d)) return S4C_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (tables) {
        qkv_prep_kernel<<<dim3(B, ceil_div(T, kQkPrepNodes)), 128, 0, stream>>>(cache_len, parent, n_nodes, position_base, T, C, d, (double)rope_theta, row_base, rope, status);
        S4C_RETURN_IF_CUDA_ERROR();
    }
    static bool configured[64] = {};  // the dynamic shared memory opt-in is per device
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return S4C_ERR_CUDA;
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(qkv_rope_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kQkSmemBytes) != cudaSuccess) {
            cudaGetLastError();
            return S4C_ERR_CUDA;
        }
        configured[dev] = true;
    }
    QkParams prm;
    prm.R = R, prm.T = T, prm.Hq = Hq, prm.Hkv = Hkv, prm.d = d, prm.C = C, prm.k_steps = H / kQkBK;
    prm.x_rows = x_rows, prm.stages = stages;
    prm.row_base = row_base, prm.rope = rope;
    prm.q_out = static_cast<__nv_bfloat16*>(q_out), prm.k_cache = static_cast<__nv_bfloat16*>(k_cache);
    prm.v_cache = static_cast<__nv_bfloat16*>(v_cache), prm.status = status;
    prm.wait_x = tables ? 0 : 1;
    cudaLaunchAttribute pdl;
    pdl.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.stream = stream, cfg.attrs = &pdl, cfg.numAttrs = 1;
    cfg.gridDim = dim3(heads, ceil_div(R, kQkBM), 1), cfg.blockDim = dim3(kQkThreads, 1, 1);
    cfg.dynamicSmemBytes = kQkSmemBytes;
    if (cudaLaunchKernelEx(&cfg, qkv_rope_kernel, map_x, map_w, prm) != cudaSuccess) {
        cudaGetLastError();
        return S4C_ERR_CUDA;
    }
    return S4C_OK;
}
}  // namespace s4c

extern "C" s4c_status s4c_qkv_rope(const void* x, const void* w_qkv, const int32_t* cache_len, const int32_t* parent,
                                   const int32_t* n_nodes, void* q_out, void* k_cache, void* v_cache, int B, int T, int H,
                                   int Hq, int Hkv, int d, int C, float rope_theta, int32_t* status, void* workspace,
                                   size_t workspace_bytes, s4c_stream_t stream) {
    return s4c::qk_run(true, x, w_qkv, cache_len, parent, n_nodes, nullptr, q_out, k_cache, v_cache, B, T, H, Hq, Hkv, d, C, rope_theta,
                       status, workspace, workspace_bytes, stream);
}

extern "C" s4c_status s4c_qkv_rope_at(const void* x, const void* w_qkv, const int32_t* cache_len, const int32_t* position_base,
                                      const int32_t* parent, const int32_t* n_nodes, void* q_out, void* k_cache, void* v_cache,
                                      int B, int T, int H, int Hq, int Hkv, int d, int C, float rope_theta, int32_t* status,
                                      void* workspace, size_t workspace_bytes, s4c_stream_t stream) {
    if (!position_base) return S4C_ERR_NULL;
    return s4c::qk_run(true, x, w_qkv, cache_len, parent, n_nodes, position_base, q_out, k_cache, v_cache, B, T, H, Hq, Hkv, d, C,
                       rope_theta, status, workspace, workspace_bytes, stream);
}

extern "C" s4c_status s4c_qkv_rope_same_tree(const void* x, const void* w_qkv, void* q_out, void* k_cache, void* v_cache, int B,
                                             int T, int H, int Hq, int Hkv, int d, int C, int32_t* status, void* workspace,
                                             size_t workspace_bytes, s4c_stream_t stream) {
    return s4c::qk_run(false, x, w_qkv, nullptr, nullptr, nullptr, nullptr, q_out, k_cache, v_cache, B, T, H, Hq, Hkv, d, C, 10000.f, status,
                       workspace, workspace_bytes, stream);
}
