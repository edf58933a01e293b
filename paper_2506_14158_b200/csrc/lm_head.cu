// s4c_lm_head_greedy: the LM head of the verify pass fused with the greedy choice (Eq. 6: t = Argmax(LM_head(f));
// Section 3.2: the target's logits at every node of the tree; Section 4.1: greedy decoding) -- the [rows, V] logits are
// never written to memory.  s4c_tree_accept_tokens: the greedy walk of the tree on those choices.
//
// logits[r, v] = sum_h hidden[r, h] * weight[v, h] is a dense contraction: bf16 operands on the tcgen05 tensor cores, f32
// accumulators in tensor memory.  One persistent CTA per SM walks over 128-token tiles of the vocabulary (tile = CTA index,
// + grid size, ...): every weight tile leaves HBM once and meets all rows (up to 256: two 128-row accumulators side by
// side on one weight stream); the hidden states (a few MB) are re-read from L2.  Roles: warp 0 requests tiles by TMA
// (64-element K slices, 128-byte swizzle, a ring of 192 KB cut into 4 to 12 stages), warp 1 issues the products and commits them to the
// ring's "empty" barriers and to the accumulator's "full" barrier, warps 2-5 read a finished accumulator (one row per
// thread), keep the running (maximum, first token that reaches it) per row across the CTA's tiles while the next tile's
// products fill the other accumulator.  A second small kernel merges the CTAs' candidates per row (greater logit, then
// lower token).  Every wait on a barrier is bounded; a CTA that gives up waits for what it set in motion, frees its
// tensor memory and flags the call.
#include <cuda.h>
#include <limits.h>
#include <math.h>

#include <algorithm>

#include "s4c_common.cuh"
#include "tc_primitives.cuh"

namespace s4c {

using namespace tcp;

constexpr int kLmBM = 128;        // rows per accumulator (tensor-memory lanes)
constexpr int kLmBK = 64;         // hidden elements per stage (one 128-byte swizzled row)
constexpr int kLmTileBytes = kLmBM * kLmBK * 2;  // 16 KB: one 128 x 64 bf16 operand tile
constexpr int kLmThreads = 192;   // producer warp, issuer warp, four epilogue warps
constexpr int kLmRowsPerLaunch = 2 * kLmBM;

// Vocabulary entries per tile: a launch-time choice (a multiple of 32), so that the tiles spread evenly over the CTAs
// (V = 32000 on 148 SMs: 143 tiles of 224 instead of 250 of 128 in two uneven rounds).  Two row tiles leave room for 128.
template <int NM>
struct LmCfg {
    static constexpr int kMaxBN = NM == 2 ? 128 : 256;
    static constexpr int kRingBytes = 192 * 1024;      // cut into stages at launch: a stage holds the rows and tokens that exist
    static constexpr int kMaxStages = 12;
    static constexpr int kTmemCols = 2 * NM * kMaxBN;  // two accumulator buffers: all 512 columns
    static constexpr int kBars = 2 * kMaxStages + 5;   // full[], empty[], acc_full[2], acc_empty[2], drain
    static constexpr int kSmemBytes = 1024 + kRingBytes + kBars * 8 + 16;
};

struct LmParams {
    int rows;        // rows of this launch (<= 256), starting at row0 of the hidden states
    int row0;
    int V;
    int bn;          // vocabulary entries per tile
    int a_rows;      // rows of a hidden-state box (a multiple of 32, <= 128): 26 rows need not move 128
    int stages;      // ring stages of a_rows * NM + bn rows of 128 bytes each
    int k_steps;     // H / 64
    float* part_v;   // [grid][256][KT] the CTAs' best logits per row, best first
    int32_t* part_t; // [grid][256][KT] and their tokens
    int32_t* status; // one word (may be null): S4C_SEQ_TIMEOUT is OR-ed in when a wait was given up
};

template <int NM, int KT>
__global__ void __launch_bounds__(kLmThreads, 1)
lm_head_greedy_kernel(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_w, const LmParams prm) {
    using Cfg = LmCfg<NM>;
    constexpr int SM = Cfg::kMaxStages;
    const int S = prm.stages;
    const int a_bytes = prm.a_rows * kLmBK * 2, stage_bytes = NM * a_bytes + prm.bn * kLmBK * 2;
    extern __shared__ unsigned char lm_smem_raw[];
    const uint32_t raw = smem_u32(lm_smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // swizzled tiles start on 1024-byte boundaries
    unsigned char* gen = lm_smem_raw + (base - raw);
    const uint32_t bars = base + Cfg::kRingBytes;
    auto FULL = [&](int s) { return bars + 8u * s; };
    auto EMPTY = [&](int s) { return bars + 8u * (SM + s); };
    auto ACC_FULL = [&](int b) { return bars + 8u * (2 * SM + b); };
    auto ACC_EMPTY = [&](int b) { return bars + 8u * (2 * SM + 2 + b); };
    const uint32_t DRAIN = bars + 8u * (2 * SM + 4);
    volatile int* tail = reinterpret_cast<volatile int*>(gen + Cfg::kRingBytes + Cfg::kBars * 8);
    volatile int* tmem_slot = tail;       // written by tcgen05.alloc
    volatile int* dead = tail + 1;        // a wait was given up
    volatile int* issued_s = tail + 2;    // stage fills the producer has requested
    auto sA = [&](int s, int t) { return base + s * stage_bytes + t * a_bytes; };
    auto sB = [&](int s) { return base + s * stage_bytes + NM * a_bytes; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bn = prm.bn;
    const int n_tiles = (prm.V + bn - 1) / bn;
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) mbar_init(FULL(s), 1), mbar_init(EMPTY(s), 1);
        for (int b = 0; b < 2; ++b) mbar_init(ACC_FULL(b), 1), mbar_init(ACC_EMPTY(b), 4);
        mbar_init(DRAIN, 1);
        mbar_fence_init();
        *dead = 0, *issued_s = 0;
        tma_prefetch_desc(&map_h), tma_prefetch_desc(&map_w);
    }
    if (warp == 1) tmem_alloc(smem_u32(const_cast<int*>(tmem_slot)), Cfg::kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = (uint32_t)*tmem_slot;
    auto TM = [&](int buf, int t) { return tmem + (uint32_t)((buf * NM + t) * Cfg::kMaxBN); };

    if (warp == 0) {
        // ================= producer: hidden-state and weight tiles into the ring =================
        if (lane == 0) {
            int fill = 0, s = 0;
            uint32_t ph = 0;  // the ring pass's parity (stage and parity are stepped, not divided out: S is not a constant)
            bool ok = true;
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x)
                for (int ks = 0; ks < prm.k_steps; ++ks, ++fill, s = s + 1 == S ? 0 : s + 1, ph ^= (s == 0)) {
                    ok = mbar_wait(EMPTY(s), ph ^ 1, dead);
                    if (!ok) break;
                    mbar_expect_tx(FULL(s), stage_bytes);
#pragma unroll
                    for (int t = 0; t < NM; ++t) tma_load_2d(sA(s, t), &map_h, FULL(s), ks * kLmBK, prm.row0 + t * kLmBM);
                    tma_load_2d(sB(s), &map_w, FULL(s), ks * kLmBK, tile * bn);
                }
            *issued_s = fill;
        }
        __syncwarp();
    } else if (warp == 1) {
        // ================= issuer: acc[t] = hidden tile t x weight tile^T over all K slices =================
        if (lane == 0) {
            const uint32_t idesc = instr_desc_bf16(kLmBM, bn, false);
            int it = 0, s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++it) {
                const int buf = it & 1;
                ok = mbar_wait(ACC_EMPTY(buf), ((it >> 1) & 1) ^ 1, dead);  // the epilogue has read this buffer
                for (int ks = 0; ks < prm.k_steps && ok; ++ks, s = s + 1 == S ? 0 : s + 1, ph ^= (s == 0)) {
                    ok = mbar_wait(FULL(s), ph, dead);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t b_desc = smem_desc_sw128(sB(s), 16, 1024);
#pragma unroll
                    for (int t = 0; t < NM; ++t) {
                        const uint64_t a_desc = smem_desc_sw128(sA(s, t), 16, 1024);
#pragma unroll
                        for (int kk = 0; kk < kLmBK / 16; ++kk)  // 32 bytes per K step inside the swizzled row (field unit: 16 B)
                            tc_mma_bf16(TM(buf, t), a_desc + 2u * kk, b_desc + 2u * kk, idesc, (ks > 0 || kk > 0) ? 1u : 0u);
                    }
                    tc_commit(EMPTY(s));  // the stage is free once these products have read it
                }
                if (ok) tc_commit(ACC_FULL(buf));
            }
        }
        __syncwarp();
    } else {
        // ================= epilogue: running (maximum, first token) per row over this CTA's tiles =================
        const int q = warp & 3;  // the tensor-memory lanes this warp may read: 32 q .. 32 q + 31
        float best_v[NM][KT];  // the KT best of the row so far, best first; equal logits: the lower token first
        int best_t[NM][KT];
#pragma unroll
        for (int t = 0; t < NM; ++t)
#pragma unroll
            for (int j = 0; j < KT; ++j) best_v[t][j] = -INFINITY, best_t[t][j] = INT_MAX;
        int it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++it) {
            const int buf = it & 1;
            ok = mbar_wait(ACC_FULL(buf), (it >> 1) & 1, dead);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const int col0 = tile * bn;
#pragma unroll
            for (int t = 0; t < NM; ++t) {
#pragma unroll
                for (int c = 0; c < Cfg::kMaxBN / 32; ++c) {
                    if (c * 32 >= bn) break;
                    uint32_t r[32];
                    tmem_ld32(TM(buf, t) + ((uint32_t)(q * 32) << 16) + c * 32, r);
                    tmem_wait_ld();
                    if (KT == 1) {
                        // one candidate per row: compare and keep (tokens ascend within a CTA and the comparison is strict:
                        // of equal logits the lower token stays)
                        // (most runs of 32 hold nothing above the row's maximum so far: one maximum over the run settles that)
                        float run_max = -INFINITY;
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (col0 + c * 32 + j < prm.V) run_max = fmaxf(run_max, __uint_as_float(r[j]));
                        if (run_max > best_v[t][0]) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                const float v = __uint_as_float(r[j]);
                                const int col = col0 + c * 32 + j;
                                if (col < prm.V && v > best_v[t][0]) best_v[t][0] = v, best_t[t][0] = col;
                            }
                        }
                    } else {
                        // a ranked list per row: which of the 32 logits beat the list's last entry is one bit each; only
                        // those (a few per run once the list has settled) are looked at again, in token order, and enter by
                        // strict comparisons, so that of equal logits the lower token stays ahead.  NaN and columns past
                        // the vocabulary never enter.  (The values are indexed by a run-time bit position: the compiler
                        // keeps this copy in local memory, which the L1 serves.)
                        float lv[32];
                        uint32_t m = 0;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            lv[j] = __uint_as_float(r[j]);
                            m |= (col0 + c * 32 + j < prm.V && lv[j] > best_v[t][KT - 1]) ? (1u << j) : 0u;
                        }
                        while (m) {
                            const int j = __ffs(m) - 1;
                            m &= m - 1;
                            const float v = lv[j];
                            if (v > best_v[t][KT - 1]) {
                                best_v[t][KT - 1] = v, best_t[t][KT - 1] = col0 + c * 32 + j;
#pragma unroll
                                for (int jj = KT - 1; jj > 0; --jj)
                                    if (best_v[t][jj] > best_v[t][jj - 1]) {
                                        const float fv = best_v[t][jj];
                                        best_v[t][jj] = best_v[t][jj - 1], best_v[t][jj - 1] = fv;
                                        const int ft = best_t[t][jj];
                                        best_t[t][jj] = best_t[t][jj - 1], best_t[t][jj - 1] = ft;
                                    }
                            }
                        }
                    }
                    __syncwarp();  // the lanes took different ways through the run; the next tensor-memory load is warp-wide
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(ACC_EMPTY(buf));
        }
#pragma unroll
        for (int t = 0; t < NM; ++t) {
            const int r = t * kLmBM + q * 32 + lane;
#pragma unroll
            for (int j = 0; j < KT; ++j) {
                prm.part_v[((size_t)blockIdx.x * kLmRowsPerLaunch + r) * KT + j] = best_v[t][j];
                prm.part_t[((size_t)blockIdx.x * kLmRowsPerLaunch + r) * KT + j] = best_t[t][j];
            }
        }
    }
    griddep_launch_dependents();
    __syncthreads();
    if (*dead) {
        // a wait was given up: nothing more is issued; what is still in flight lands before shared and tensor memory go
        if (threadIdx.x == 0) {
            const int issued = *issued_s;
            for (int s = 0; s < S; ++s) {
                int last = -1;  // the last fill requested into stage s
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
        tmem_dealloc(tmem, Cfg::kTmemCols);
    }
}

// Per row: the k best of the CTAs' candidates, best first (greater logit, then lower token).  One warp per row: the
// candidates (at most 1024 CTAs x 8) come into shared memory once -- independent loads, in flight together --, then round j
// takes the best candidate that ranks after round j-1's (the candidates' tokens are distinct).
constexpr int kLmMergeRows = 4;      // rows (warps) per CTA
constexpr int kLmMergeStage = 1184;  // candidates staged per row: 148 CTAs x 8; beyond that the rounds read global memory
__global__ void __launch_bounds__(kLmMergeRows * 32)
lm_head_merge_kernel(const float* __restrict__ part_v, const int32_t* __restrict__ part_t, int n_parts, int kt, int rows, int k,
                     int32_t* __restrict__ token, float* __restrict__ logit) {
    __shared__ float sv[kLmMergeRows][kLmMergeStage];
    __shared__ int st[kLmMergeRows][kLmMergeStage];
    griddep_wait();
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = blockIdx.x * kLmMergeRows + w;
    if (r >= rows) return;
    const int total = n_parts * kt;  // candidate c: CTA c / kt, rank c % kt
    const bool staged = total <= kLmMergeStage;
    auto at = [&](int c) { return ((size_t)(c / kt) * kLmRowsPerLaunch + r) * kt + (c % kt); };
    if (staged) {
        for (int c = lane; c < total; c += 32) sv[w][c] = part_v[at(c)], st[w][c] = part_t[at(c)];
        __syncwarp();
    }
    float pv = INFINITY;
    int pt = -1;
    for (int j = 0; j < k; ++j) {
        float bv = -INFINITY;
        int bt = INT_MAX;
        for (int c = lane; c < total; c += 32) {
            const float v = staged ? sv[w][c] : part_v[at(c)];
            const int t = staged ? st[w][c] : part_t[at(c)];
            const bool after = v < pv || (v == pv && t > pt);
            if (t != INT_MAX && after && (v > bv || (v == bv && t < bt))) bv = v, bt = t;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int ot = __shfl_xor_sync(0xffffffffu, bt, o);
            if (ov > bv || (ov == bv && ot < bt)) bv = ov, bt = ot;
        }
        pv = bv, pt = bt;
        if (lane == 0) {
            token[(size_t)r * k + j] = bt == INT_MAX ? -1 : bt;  // fewer than k comparable logits in the row (k > V, NaN)
            if (logit) logit[(size_t)r * k + j] = bt == INT_MAX ? -INFINITY : bv;
        }
        if (bt == INT_MAX) pv = -INFINITY, pt = INT_MAX;  // nothing ranks after "none"
    }
}

// ----------------------------------------------------------------------------- greedy walk on known choices
struct TokWalkShared {
    int32_t par[S4C_MAX_T];
    int32_t tok[S4C_MAX_T];
    int32_t tgt[S4C_MAX_T];
    int depth[S4C_MAX_T];
    uint32_t anc[S4C_MAX_T][S4C_MASK_WORDS];
    int flag;
};

__global__ void __launch_bounds__(128)
accept_tokens_kernel(const int32_t* __restrict__ target_token, const int32_t* __restrict__ tokens,
                     const int32_t* __restrict__ parent, const int32_t* __restrict__ n_nodes, int T, int V, int max_depth,
                     int32_t* __restrict__ accept_len, int32_t* __restrict__ path, int32_t* __restrict__ next_token,
                     int32_t* __restrict__ status) {
    __shared__ TokWalkShared sh;
    const int b = blockIdx.x, tid = threadIdx.x;
    const int n = n_nodes ? n_nodes[b] : T;
    int32_t* pth = path + (size_t)b * (max_depth + 1);
    for (int i = tid; i < T; i += blockDim.x) {
        sh.par[i] = parent[(size_t)b * T + i];
        sh.tok[i] = tokens[(size_t)b * T + i];
        sh.tgt[i] = target_token[(size_t)b * T + i];
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
    if (tid != 0) return;
    // a node is accepted when every node on its path carries the target's choice at its parent; parents come first, so
    // one pass in index order settles all nodes (at most 128): reuse the depth array's sign for "accepted"
    int end = 0;
    for (int i = 1; i < n; ++i) {
        const int p = sh.par[i];
        const bool ok = sh.depth[p] >= 0 && sh.tok[i] == sh.tgt[p];
        if (!ok)
            sh.depth[i] = -1 - sh.depth[i];  // not accepted (depth kept, negated)
        else if (sh.depth[i] > sh.depth[end])
            end = i;  // the deepest accepted node, the lowest index among equals
    }
    for (int j = 0; j <= max_depth; ++j) pth[j] = -1;
    for (int t = end; t >= 0; t = sh.par[t]) pth[sh.depth[t]] = t;
    accept_len[b] = sh.depth[end];
    next_token[b] = sh.tgt[end];
}

// ----------------------------------------------------------------------------- host side
typedef CUresult (*LmEncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                    const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static LmEncodeTiledFn lm_encode_fn() {
    static LmEncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<LmEncodeTiledFn>(p);
    }
    return fn;
}

// [rows, H] bf16 row-major, boxes of box_rows rows x 64 elements (128 bytes), 128-byte swizzle, zero fill out of range
static bool lm_make_map(CUtensorMap* map, const void* ptr, uint64_t rows, int H, int box_rows) {
    LmEncodeTiledFn fn = lm_encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)H, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)H * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kLmBK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static int lm_sm_count() {
    static int n = 0;
    if (!n) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
            cudaGetLastError();
            n = 148;
        }
    }
    return n;
}

static inline int lm_kt(int k) { return k <= 1 ? 1 : (k <= 4 ? 4 : 8); }  // candidates a thread keeps per row
static inline size_t lm_ws_layout(int V, int k, char* base, float** part_v, int32_t** part_t) {
    const size_t parts = (size_t)std::min(ceil_div(V, 64), 1024);  // at most one CTA per tile (64 entries or more), never more than this
    size_t off = 0;
    if (part_v) *part_v = reinterpret_cast<float*>(base + off);
    off += round_up(parts * kLmRowsPerLaunch * lm_kt(k) * sizeof(float), 256);
    if (part_t) *part_t = reinterpret_cast<int32_t*>(base + off);
    off += round_up(parts * kLmRowsPerLaunch * lm_kt(k) * sizeof(int32_t), 256);
    return off;
}

template <int NM, int KT>
static s4c_status lm_launch(const CUtensorMap& map_h, const CUtensorMap& map_w, const LmParams& prm, int grid, cudaStream_t stream) {
    using Cfg = LmCfg<NM>;
    if (cudaFuncSetAttribute(lm_head_greedy_kernel<NM, KT>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes) !=
        cudaSuccess) {
        cudaGetLastError();
        return S4C_ERR_CUDA;
    }
    lm_head_greedy_kernel<NM, KT><<<grid, kLmThreads, Cfg::kSmemBytes, stream>>>(map_h, map_w, prm);
    S4C_RETURN_IF_CUDA_ERROR();
    return S4C_OK;
}

}  // namespace s4c

extern "C" size_t s4c_lm_head_topk_workspace_bytes(int R, int V, int H, int k) {
    if (R < 1 || V < 1 || H < 1 || k < 1 || k > 8) return 0;
    return s4c::lm_ws_layout(V, k, nullptr, nullptr, nullptr);
}

extern "C" s4c_status s4c_lm_head_topk(const void* hidden, const void* weight, int R, int V, int H, int k, int32_t* token,
                                       float* logit, int32_t* status, void* workspace, size_t workspace_bytes,
                                       s4c_stream_t stream_) {
    using namespace s4c;
    if (!hidden || !weight || !token) return S4C_ERR_NULL;
    if (R < 0 || V < 1 || H < kLmBK || H % kLmBK != 0 || k < 1) return S4C_ERR_SHAPE;
    if (k > 8) return S4C_ERR_UNSUPPORTED;
    if (!aligned16(hidden) || !aligned16(weight)) return S4C_ERR_ALIGN;
    if (R == 0) return S4C_OK;
    float* part_v;
    int32_t* part_t;
    const size_t need = lm_ws_layout(V, k, nullptr, nullptr, nullptr);
    if (!workspace || workspace_bytes < need || !aligned256(workspace)) return S4C_ERR_WORKSPACE;
    lm_ws_layout(V, k, static_cast<char*>(workspace), &part_v, &part_t);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (status && cudaMemsetAsync(status, 0, sizeof(int32_t), stream) != cudaSuccess) {
        cudaGetLastError();
        return S4C_ERR_CUDA;
    }
    const int sms = std::min(lm_sm_count(), 1024), kt = lm_kt(k);
    // groups of up to 256 rows; each group streams the weights once
    for (int row0 = 0; row0 < R; row0 += kLmRowsPerLaunch) {
        LmParams prm;
        prm.rows = std::min(kLmRowsPerLaunch, R - row0), prm.row0 = row0, prm.V = V, prm.k_steps = H / kLmBK;
        prm.part_v = part_v, prm.part_t = part_t, prm.status = status;
        // tile width: the one that costs the fewest (rounds of tiles over the CTAs) x (entries per tile)
        prm.bn = 128;
        if (prm.rows <= kLmBM) {
            long long best = -1;
            for (int bn = 64; bn <= LmCfg<1>::kMaxBN; bn += 32) {
                const long long cost = (long long)ceil_div(ceil_div(V, bn), sms) * bn;
                if (best < 0 || cost <= best) best = cost, prm.bn = bn;
            }
        }
        const int grid = std::min(ceil_div(V, prm.bn), sms);
        const bool two = prm.rows > kLmBM;
        // the ring: a stage holds one K slice of the rows that exist (a box of 26 rows moves 32, not 128) and of the tile's
        // tokens; as many stages as fit.  The product always reads 128 rows from a stage's start: one spare tile at the
        // ring's end keeps that read inside the ring when a stage is shorter than a full tile.
        prm.a_rows = two ? kLmBM : std::min(kLmBM, (int)round_up((size_t)prm.rows, 32));
        const int stage_bytes = (two ? 2 : 1) * prm.a_rows * kLmBK * 2 + prm.bn * kLmBK * 2;
        prm.stages = std::min(LmCfg<1>::kMaxStages, (LmCfg<1>::kRingBytes - (prm.a_rows < kLmBM ? kLmTileBytes : 0)) / stage_bytes);
        CUtensorMap map_h, map_w;
        if (!lm_make_map(&map_h, hidden, (uint64_t)R, H, prm.a_rows) || !lm_make_map(&map_w, weight, (uint64_t)V, H, prm.bn))
            return S4C_ERR_CUDA;
        const s4c_status st = kt == 1   ? (two ? lm_launch<2, 1>(map_h, map_w, prm, grid, stream) : lm_launch<1, 1>(map_h, map_w, prm, grid, stream))
                              : kt == 4 ? (two ? lm_launch<2, 4>(map_h, map_w, prm, grid, stream) : lm_launch<1, 4>(map_h, map_w, prm, grid, stream))
                                        : (two ? lm_launch<2, 8>(map_h, map_w, prm, grid, stream) : lm_launch<1, 8>(map_h, map_w, prm, grid, stream));
        if (st != S4C_OK) return st;
        cudaLaunchAttribute pdl;
        pdl.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        pdl.val.programmaticStreamSerializationAllowed = 1;
        cudaLaunchConfig_t cfg = {};
        cfg.stream = stream, cfg.attrs = &pdl, cfg.numAttrs = 1;
        cfg.gridDim = dim3(ceil_div(prm.rows, kLmMergeRows), 1, 1), cfg.blockDim = dim3(kLmMergeRows * 32, 1, 1);  // a warp per row
        if (cudaLaunchKernelEx(&cfg, lm_head_merge_kernel, (const float*)part_v, (const int32_t*)part_t, grid, kt, prm.rows, k,
                               token + (size_t)row0 * k, logit ? logit + (size_t)row0 * k : (float*)nullptr) != cudaSuccess) {
            cudaGetLastError();
            return S4C_ERR_CUDA;
        }
    }
    return S4C_OK;
}

extern "C" size_t s4c_lm_head_greedy_workspace_bytes(int R, int V, int H) { return s4c_lm_head_topk_workspace_bytes(R, V, H, 1); }

extern "C" s4c_status s4c_lm_head_greedy(const void* hidden, const void* weight, int R, int V, int H, int32_t* token,
                                         float* max_logit, int32_t* status, void* workspace, size_t workspace_bytes,
                                         s4c_stream_t stream_) {
    return s4c_lm_head_topk(hidden, weight, R, V, H, 1, token, max_logit, status, workspace, workspace_bytes, stream_);
}

extern "C" s4c_status s4c_tree_accept_tokens(const int32_t* target_token, const int32_t* tokens, const int32_t* parent,
                                             const int32_t* n_nodes, int B, int T, int V, int max_depth, int32_t* accept_len,
                                             int32_t* path, int32_t* next_token, int32_t* status, s4c_stream_t stream_) {
    using namespace s4c;
    if (!target_token || !tokens || !parent || !accept_len || !path || !next_token) return S4C_ERR_NULL;
    if (B < 0 || T < 1 || T > S4C_MAX_T || V < 1 || max_depth < 0 || max_depth >= S4C_MAX_T) return S4C_ERR_SHAPE;
    if (B == 0) return S4C_OK;
    accept_tokens_kernel<<<B, 128, 0, static_cast<cudaStream_t>(stream_)>>>(target_token, tokens, parent, n_nodes, T, V, max_depth,
                                                                           accept_len, path, next_token, status);
    S4C_RETURN_IF_CUDA_ERROR();
    return S4C_OK;
}
