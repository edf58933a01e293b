// Tree-masked attention on the 5th-generation tensor cores (Section 3.2 tree mask; Figure 3) for bf16 caches.
//
// One CTA = one KV head of one sequence x one tile of 128 query rows x one split of the cache.  The query
// rows of the G = Hq/Hkv heads that share the KV head are packed into the MMA M dimension (row = g*T + node),
// so K/V stream from HBM once per KV head.  Warp-specialised:
//   warp 0      TMA producer: Q once, then K and V tiles of 64 slots into 128B-swizzled shared-memory rings
//   warp 1      MMA issuer: S = Q K^T (tcgen05.mma kind::f16, M128 N64 K16 x d/16) into one of two TMEM
//               score buffers, O += P V (M128 N=d K16 x 4) into a TMEM accumulator; owns the TMEM allocation
//   warps 2..5  one thread per query row: tcgen05.ld of the scores, tree / tail masking from the per-node
//               ancestor bitmask, online softmax in fp32 (base-2), rescale of O in TMEM when the running max
//               moves, P rounded to bf16 into swizzled shared memory as the A operand of the PV product
// Partial (max, sum, unnormalised O) per split go to the workspace; the combine kernel merges them in split
// order.  Every mbarrier wait is bounded (200 ms): on expiry the CTA flags S4C_SEQ_TIMEOUT in status[b],
// stops waiting for anything else, still frees its TMEM and returns.
#include <cuda.h>
#include <math.h>

#include "s4c_common.cuh"
#include "tree_attention.cuh"

namespace s4c {

constexpr int kBM = 128;       // query rows per CTA (TMEM lanes)
constexpr int kBN = 64;        // cache slots per tile
constexpr int kTcThreads = 192;
constexpr uint64_t kWaitLimitNs = 200ull * 1000 * 1000;

template <int D>
struct TcCfg {
    static constexpr int kHalves = D / 64;                    // 64-element (128-byte) swizzle atoms along d
    static constexpr int kQBytes = kBM * D * 2;               // 32 KB (d = 128)
    static constexpr int kTileBytes = kBN * D * 2;            // 16 KB: one K or V tile
    static constexpr int kPBytes = kBM * kBN * 2;             // 16 KB
    static constexpr int kStages = D == 128 ? 4 : 6;
    static constexpr int kSmemData = kQBytes + 2 * kPBytes + 2 * kStages * kTileBytes;
    static constexpr int kNumBars = 1 + 4 * kStages + 2 + 2 + 2 + 1;
    static constexpr int kSmemBytes = 1024 /*alignment slack*/ + kSmemData + 1024 /*barriers, masks, flags*/ + S4C_MAX_T * 4 +
                                      S4C_MAX_T * S4C_MASK_WORDS * 4;
    static constexpr int kTmemCols = 256;                     // 2 x 64 score columns + up to 128 output columns
};

// ----------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait.  `dead` (shared memory) is set by the first wait that expires; later waits then give up at once.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* dead) {
    if (mbar_try_wait(bar, parity)) return;
    const uint64_t t0 = global_timer();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return;
        if (*dead) return;
        if (global_timer() - t0 > kWaitLimitNs) {
            *dead = 1;
            return;
        }
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
        "l"(map), "r"(bar), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
        "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
        "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1 (sm_100).
// Field units are 16 bytes: start address [0,14), leading byte offset [16,30), stride byte offset [32,46),
// version [46,48) = 1, layout type [61,64) = 2 (SWIZZLE_128B).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}
// Instruction descriptor, kind::f16: D = f32 (bits 4-5 = 1), A = B = bf16 (bits 7-9, 10-12 = 1), B major bit 16,
// N/8 at bits 17-22, M/16 at bits 24-28.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int M, int N, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}

struct TcParams {
    const int32_t* cache_len;
    const int32_t* parent;
    const int32_t* n_nodes;
    __nv_bfloat16* out;
    float* ws;
    int32_t* status;
    int T, Hq, Hkv, C, m_tiles, splits;
    float scale_log2;
};

// Tile range of a split: tiles are dealt out as evenly as whole tiles allow.
__device__ __forceinline__ void split_range(int n_tiles, int splits, int split, int& t0, int& t1) {
    t0 = (int)(((long long)n_tiles * split) / splits);
    t1 = (int)(((long long)n_tiles * (split + 1)) / splits);
}

template <int D>
__global__ void __launch_bounds__(kTcThreads, 1)
tree_attention_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                         const __grid_constant__ CUtensorMap map_v, const TcParams prm) {
    using Cfg = TcCfg<D>;
    constexpr int S = Cfg::kStages;
    constexpr int NH = Cfg::kHalves;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // 128B swizzle atoms need 1024-byte alignment
    unsigned char* base_ptr = smem_raw + (base - raw);
    const uint32_t sQ = base;
    const uint32_t sP = sQ + Cfg::kQBytes;
    const uint32_t sK = sP + 2 * Cfg::kPBytes;
    const uint32_t sV = sK + S * Cfg::kTileBytes;
    unsigned char* tail = base_ptr + Cfg::kSmemData;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 512);
    volatile int* dead = reinterpret_cast<volatile int*>(tail + 516);
    int* flag_s = reinterpret_cast<int*>(tail + 520);
    int32_t* par_s = reinterpret_cast<int32_t*>(tail + 1024);
    uint32_t(*anc_s)[S4C_MASK_WORDS] = reinterpret_cast<uint32_t(*)[S4C_MASK_WORDS]>(tail + 1024 + S4C_MAX_T * 4);

    const uint32_t bar0 = smem_u32(bars);
    auto BAR = [&](int i) { return bar0 + 8u * i; };
    const int Q_FULL = 0, K_FULL = 1, K_EMPTY = 1 + S, V_FULL = 1 + 2 * S, V_EMPTY = 1 + 3 * S, S_FULL = 1 + 4 * S,
              S_EMPTY = S_FULL + 2, P_FULL = S_EMPTY + 2, PV_DONE = P_FULL + 2;

    const int split = blockIdx.x, splits = prm.splits;
    const int mt = blockIdx.y % prm.m_tiles, hk = blockIdx.y / prm.m_tiles, b = blockIdx.z;
    const int T = prm.T, G = prm.Hq / prm.Hkv, R = G * T;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // ---- validate the sequence, build the ancestor bitmasks (all threads)
    const int n = prm.n_nodes ? prm.n_nodes[b] : T;
    const int L = prm.cache_len[b];
    for (int i = threadIdx.x; i < T; i += blockDim.x) par_s[i] = prm.parent[(size_t)b * T + i];
    if (threadIdx.x == 0) *dead = 0;
    __syncthreads();
    int flags = build_ancestor_masks(par_s, n, T, anc_s, nullptr, flag_s);
    if (L < 0 || (long long)L + (n > 0 ? n : 0) > (long long)prm.C) flags |= S4C_SEQ_CAPACITY;
    if (split == 0 && blockIdx.y == 0 && threadIdx.x == 0 && prm.status) prm.status[b] = flags;
    if (flags) return;

    const int Ltot = L + n;
    const int n_tiles = (Ltot + kBN - 1) / kBN;
    int t0, t1;
    split_range(n_tiles, splits, split, t0, t1);
    const int nt = t1 - t0;

    // ---- barriers and TMEM
    if (threadIdx.x == 0) {
        mbar_init(BAR(Q_FULL), 1);
        for (int s = 0; s < S; ++s) {
            mbar_init(BAR(K_FULL + s), 1), mbar_init(BAR(K_EMPTY + s), 1);
            mbar_init(BAR(V_FULL + s), 1), mbar_init(BAR(V_EMPTY + s), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(BAR(S_FULL + i), 1), mbar_init(BAR(S_EMPTY + i), 128);
            mbar_init(BAR(P_FULL + i), 128);
        }
        mbar_init(BAR(PV_DONE), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), Cfg::kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const uint32_t tmem_O = tmem + 2 * kBN;

    const int q_row0 = (b * prm.Hq + hk * G) * T + mt * kBM;  // row of the [B*Hq*T, d] view of q
    const int kv_row0 = (b * prm.Hkv + hk) * prm.C;           // row of the [B*Hkv*C, d] view of the caches

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0 && nt > 0) {
            mbar_expect_tx(BAR(Q_FULL), Cfg::kQBytes);
            for (int h = 0; h < NH; ++h) tma_load_2d(sQ + h * (kBM * 128), &map_q, BAR(Q_FULL), h * 64, q_row0);
            for (int j = 0; j < nt; ++j) {
                const int s = j % S, it = j / S, row = kv_row0 + (t0 + j) * kBN;
                mbar_wait(BAR(K_EMPTY + s), (it & 1) ^ 1, dead);
                mbar_expect_tx(BAR(K_FULL + s), Cfg::kTileBytes);
                for (int h = 0; h < NH; ++h)
                    tma_load_2d(sK + s * Cfg::kTileBytes + h * (kBN * 128), &map_k, BAR(K_FULL + s), h * 64, row);
                mbar_wait(BAR(V_EMPTY + s), (it & 1) ^ 1, dead);
                mbar_expect_tx(BAR(V_FULL + s), Cfg::kTileBytes);
                for (int h = 0; h < NH; ++h)
                    tma_load_2d(sV + s * Cfg::kTileBytes + h * (kBN * 128), &map_v, BAR(V_FULL + s), h * 64, row);
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        if (lane == 0 && nt > 0) {
            constexpr uint32_t idesc_qk = instr_desc_bf16(kBM, kBN, false);
            constexpr uint32_t idesc_pv = instr_desc_bf16(kBM, D, true);
            auto issue_pv = [&](int jj) {
                const int s = jj % S, it = jj / S;
                mbar_wait(BAR(V_FULL + s), it & 1, dead);
                mbar_wait(BAR(P_FULL + (jj & 1)), (jj >> 1) & 1, dead);
                tc_fence_after();
                const uint32_t p_base = sP + (jj & 1) * Cfg::kPBytes, v_base = sV + s * Cfg::kTileBytes;
#pragma unroll
                for (int kk = 0; kk < kBN / 16; ++kk) {
                    // A = P [128 rows][64 slots], K-major: 32 bytes per K step inside the 128-byte row
                    const uint64_t ad = smem_desc_sw128(p_base + kk * 32, 16, 1024);
                    // B = V [64 slots][d], MN-major: 16 slots (K step) = 2048 bytes; d halves kBN*128 bytes apart
                    const uint64_t bd = smem_desc_sw128(v_base + kk * 2048, kBN * 128, 1024);
                    tc_mma_bf16(tmem_O, ad, bd, idesc_pv, (jj > 0 || kk > 0) ? 1u : 0u);
                }
                tc_commit(BAR(V_EMPTY + s));
                tc_commit(BAR(PV_DONE));
            };
            mbar_wait(BAR(Q_FULL), 0, dead);
            for (int j = 0; j < nt; ++j) {
                const int s = j % S, it = j / S;
                mbar_wait(BAR(K_FULL + s), it & 1, dead);
                mbar_wait(BAR(S_EMPTY + (j & 1)), ((j >> 1) & 1) ^ 1, dead);
                tc_fence_after();
                const uint32_t k_base = sK + s * Cfg::kTileBytes;
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const int h = kk >> 2, ko = (kk & 3) * 32;  // 64-element halves along d, 32 bytes per K step
                    const uint64_t ad = smem_desc_sw128(sQ + h * (kBM * 128) + ko, 16, 1024);
                    const uint64_t bd = smem_desc_sw128(k_base + h * (kBN * 128) + ko, 16, 1024);
                    tc_mma_bf16(tmem + (j & 1) * kBN, ad, bd, idesc_qk, kk > 0 ? 1u : 0u);
                }
                tc_commit(BAR(K_EMPTY + s));
                tc_commit(BAR(S_FULL + (j & 1)));
                if (j > 0) issue_pv(j - 1);
            }
            issue_pv(nt - 1);
        }
    } else {
        // ================= softmax / correction / epilogue: one thread per query row =================
        const int wq = warp & 3;  // TMEM lane quadrant this warp may access
        const int row = wq * 32 + lane;
        const int gr = mt * kBM + row;
        const bool row_valid = gr < R;
        const int node = gr % T;
        const bool node_valid = row_valid && node < n;
        uint32_t am[S4C_MASK_WORDS];
#pragma unroll
        for (int w = 0; w < S4C_MASK_WORDS; ++w) am[w] = node_valid ? anc_s[node][w] : 0u;
        const uint32_t lane_off = (uint32_t)(wq * 32) << 16;
        const int sm_tid = threadIdx.x - 64;  // 0..127
        float m = -1e30f, l = 0.f;
        const float sc = prm.scale_log2;

        for (int j = 0; j < nt; ++j) {
            const int kv0 = (t0 + j) * kBN;
            mbar_wait(BAR(S_FULL + (j & 1)), (j >> 1) & 1, dead);
            tc_fence_after();
            uint32_t sr[2][32];
            tmem_ld32(tmem + lane_off + (j & 1) * kBN, sr[0]);
            tmem_ld32(tmem + lane_off + (j & 1) * kBN + 32, sr[1]);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(BAR(S_EMPTY + (j & 1)));

            float sv[kBN];
#pragma unroll
            for (int c = 0; c < kBN; ++c) sv[c] = __uint_as_float(sr[c >> 5][c & 31]) * sc;
            if (kv0 + kBN > L) {  // the tile touches tree slots or the tail: mask by index
#pragma unroll
                for (int c = 0; c < kBN; ++c) {
                    const int kv = kv0 + c, t = kv - L;
                    bool vis = kv < L;
                    if (!vis && t < n) vis = (am[(t >> 5) & 3] >> (t & 31)) & 1u;
                    sv[c] = vis ? sv[c] : -INFINITY;
                }
            }
            float mx = sv[0];
#pragma unroll
            for (int c = 1; c < kBN; ++c) mx = fmaxf(mx, sv[c]);
            const float m_new = row_valid ? fmaxf(m, mx) : m;
            const float alpha = exp2f(m - m_new);
            float ls = 0.f;
            uint32_t pk[kBN / 2];
#pragma unroll
            for (int c = 0; c < kBN; c += 2) {
                const float p0 = exp2f(sv[c] - m_new), p1 = exp2f(sv[c + 1] - m_new);
                ls += p0 + p1;
                const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
                pk[c >> 1] = *reinterpret_cast<const uint32_t*>(&h2);
            }
            l = l * alpha + ls;
            m = m_new;

            if (j > 0) {
                mbar_wait(BAR(PV_DONE), (j - 1) & 1, dead);
                tc_fence_after();
                if (__any_sync(0xffffffffu, row_valid && alpha != 1.f)) {
#pragma unroll
                    for (int cc = 0; cc < D / 32; ++cc) {
                        uint32_t o[32];
                        tmem_ld32(tmem_O + lane_off + cc * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
                        tmem_st32(tmem_O + lane_off + cc * 32, o);
                    }
                    tmem_wait_st();
                }
            }
            if (kv0 + kBN > Ltot) {
                // last, partial tile of the sequence: rows past the end may hold anything (even NaN); P is 0 there
                // but 0 * NaN would poison O, so those V rows are cleared before the PV product reads them
                const int s = j % S, it = j / S;
                mbar_wait(BAR(V_FULL + s), it & 1, dead);
                const int first = Ltot - kv0;  // 1..63
                unsigned char* vt = base_ptr + (sV - base) + s * Cfg::kTileBytes;
                for (int idx = sm_tid; idx < (kBN - first) * 8 * NH; idx += 128) {
                    const int h = idx / ((kBN - first) * 8), rem = idx % ((kBN - first) * 8);
                    const int r = first + rem / 8, ch = rem % 8;
                    *reinterpret_cast<uint4*>(vt + h * (kBN * 128) + r * 128 + ch * 16) = make_uint4(0, 0, 0, 0);
                }
            }
            // P row -> shared memory, K-major, 128-byte swizzle: 16-byte chunk c of row r sits at chunk c ^ (r & 7)
            {
                unsigned char* pt = base_ptr + (sP - base) + (j & 1) * Cfg::kPBytes + row * 128;
#pragma unroll
                for (int ch = 0; ch < 8; ++ch)
                    *reinterpret_cast<uint4*>(pt + ((ch ^ (row & 7)) << 4)) =
                        make_uint4(pk[4 * ch], pk[4 * ch + 1], pk[4 * ch + 2], pk[4 * ch + 3]);
            }
            fence_async_smem();
            tc_fence_before();
            mbar_arrive(BAR(P_FULL + (j & 1)));
        }

        // ---- epilogue
        if (nt > 0) {
            mbar_wait(BAR(PV_DONE), (nt - 1) & 1, dead);
            tc_fence_after();
        }
        const bool direct = splits == 1;
        const size_t orow = (size_t)(b * prm.Hq + hk * G) * T + gr;  // row of the [B*Hq*T, d] view of out
        const float inv = (node_valid && l > 0.f) ? 1.f / l : 0.f;
#pragma unroll
        for (int cc = 0; cc < D / 32; ++cc) {
            uint32_t o[32];
            if (nt > 0) {
                tmem_ld32(tmem_O + lane_off + cc * 32, o);
                tmem_wait_ld();
            } else {
#pragma unroll
                for (int c = 0; c < 32; ++c) o[c] = 0u;
            }
            if (!row_valid) continue;
            if (direct) {
                uint32_t packed[16];
#pragma unroll
                for (int c = 0; c < 32; c += 2) {
                    const __nv_bfloat162 h2 =
                        __floats2bfloat162_rn(__uint_as_float(o[c]) * inv, __uint_as_float(o[c + 1]) * inv);
                    packed[c >> 1] = *reinterpret_cast<const uint32_t*>(&h2);
                }
                uint4* dst = reinterpret_cast<uint4*>(prm.out + orow * D + cc * 32);
#pragma unroll
                for (int v = 0; v < 4; ++v)
                    dst[v] = make_uint4(packed[4 * v], packed[4 * v + 1], packed[4 * v + 2], packed[4 * v + 3]);
            } else {
                float* w = prm.ws + (orow * splits + split) * (D + 2) + cc * 32;
                if (!node_valid) {
#pragma unroll
                    for (int c = 0; c < 32; ++c) o[c] = 0u;
                }
#pragma unroll
                for (int c = 0; c < 32; c += 2)
                    *reinterpret_cast<float2*>(w + c) = make_float2(__uint_as_float(o[c]), __uint_as_float(o[c + 1]));
            }
        }
        if (!direct && row_valid) {
            float* w = prm.ws + (orow * splits + split) * (D + 2) + D;
            *reinterpret_cast<float2*>(w) = make_float2(node_valid ? m : -INFINITY, node_valid ? l : 0.f);
        }
        tc_fence_before();
    }

    __syncthreads();
    if (threadIdx.x == 0 && *dead && prm.status) atomicOr(prm.status + b, S4C_SEQ_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, Cfg::kTmemCols);
    }
}

// ----------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// [rows, d] bf16 row-major, boxes of box_rows x 64 elements (128 bytes), 128-byte swizzle, zero fill out of range
static bool make_map(CUtensorMap* map, const void* ptr, uint64_t rows, int d, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)d * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool tc_supported(int T, int Hq, int Hkv, int d, s4c_dtype dt) { return dt == S4C_BF16 && (d == 128 || d == 64); }

int tc_m_tiles(int T, int Hq, int Hkv) { return ceil_div((Hq / Hkv) * T, kBM); }

int tc_splits(int B, int T, int Hq, int Hkv, int C) {
    const int base = B * Hkv * tc_m_tiles(T, Hq, Hkv);
    int s = 148 / base;  // one resident CTA per SM: fill one wave
    const int max_by_len = ceil_div(C, kBN) / 2;  // at least two tiles per split
    if (s > max_by_len) s = max_by_len;
    if (s > 64) s = 64;
    return s < 1 ? 1 : s;
}

size_t tc_workspace_bytes(int B, int T, int Hq, int Hkv, int d, int C) {
    const int s = tc_splits(B, T, Hq, Hkv, C);
    return s == 1 ? 0 : round_up((size_t)B * Hq * T * s * (d + 2) * sizeof(float), 256);
}

template <int D>
static s4c_status launch_tc(const void* q, const void* k, const void* v, const TcParams& prm, int B, cudaStream_t stream) {
    using Cfg = TcCfg<D>;
    static bool configured[64] = {};  // the opt-in to > 48 KB of dynamic shared memory is per device
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return S4C_ERR_CUDA;
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(tree_attention_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 Cfg::kSmemBytes) != cudaSuccess)
            return S4C_ERR_CUDA;
        configured[dev] = true;
    }
    CUtensorMap mq, mk, mv;
    if (!make_map(&mq, q, (uint64_t)B * prm.Hq * prm.T, D, kBM) ||
        !make_map(&mk, k, (uint64_t)B * prm.Hkv * prm.C, D, kBN) ||
        !make_map(&mv, v, (uint64_t)B * prm.Hkv * prm.C, D, kBN))
        return S4C_ERR_CUDA;
    dim3 grid(prm.splits, prm.m_tiles * prm.Hkv, B);
    tree_attention_tc_kernel<D><<<grid, kTcThreads, Cfg::kSmemBytes, stream>>>(mq, mk, mv, prm);
    S4C_RETURN_IF_CUDA_ERROR();
    return S4C_OK;
}

s4c_status tree_attention_tc(const void* q, const void* k, const void* v, const int32_t* cache_len,
                             const int32_t* parent, const int32_t* n_nodes, void* out, int B, int T, int Hq, int Hkv,
                             int d, int C, float scale, int32_t* status, void* ws, cudaStream_t stream) {
    TcParams prm;
    prm.cache_len = cache_len, prm.parent = parent, prm.n_nodes = n_nodes;
    prm.out = static_cast<__nv_bfloat16*>(out), prm.ws = static_cast<float*>(ws), prm.status = status;
    prm.T = T, prm.Hq = Hq, prm.Hkv = Hkv, prm.C = C;
    prm.m_tiles = tc_m_tiles(T, Hq, Hkv);
    prm.splits = tc_splits(B, T, Hq, Hkv, C);
    prm.scale_log2 = scale * 1.4426950408889634f;
    s4c_status st = d == 128 ? launch_tc<128>(q, k, v, prm, B, stream) : launch_tc<64>(q, k, v, prm, B, stream);
    if (st != S4C_OK) return st;
    if (prm.splits > 1) return tree_attention_combine(ws, cache_len, parent, n_nodes, out, B, T, Hq, d, C, prm.splits, S4C_BF16, stream);
    return S4C_OK;
}

}  // namespace s4c
