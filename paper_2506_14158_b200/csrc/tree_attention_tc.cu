// Tree-masked attention on the 5th-generation tensor cores (Section 3.2 tree mask; Figure 3) for bf16 caches.
//
// One CTA = one KV head of one sequence x NM tiles of 128 query rows x one split of the cache.  The query
// rows of the G = Hq/Hkv heads that share the KV head are packed into the MMA M dimension (row = g*T + node),
// so K/V stream from HBM once per KV head (NM = 2 covers G*T up to 256 rows, the GQA case, with one pass).
// Warp-specialised:
//   warp 0        TMA producer: Q once, then K and V tiles of 64 slots into 128B-swizzled shared-memory rings
//   next NM + 1   MMA issuers (the loops run warp-uniformly, so that descriptors stay in uniform registers; an
//                 elected lane issues): one QK issuer warp per row tile sends S = Q K^T (tcgen05.mma kind::f16,
//                 M128 N64 K16 x d/16) into one of the TMEM score buffers of its row tile, one PV issuer warp sends
//                 O += P V (M128 N=d K16 x 4, P read from tensor memory) into each row tile's TMEM accumulator;
//                 warp 1 owns the TMEM allocation
//   then          one group of four warps per row tile, one thread per query row: tcgen05.ld of the scores,
//                 tree / tail masking from the row's ancestor bitmask (built from parent[] by the thread
//                 itself), online softmax in fp32 (base 2; the running offset only moves when the maximum
//                 grew by more than 2^8, so O in TMEM is rarely rescaled), P rounded to bf16 back into the score
//                 buffer in tensor memory, the A operand of the PV product
// Split-KV without a second launch: the splits of one (sequence, KV head, row-tile group) form a thread-block
// cluster; every CTA parks its partial (offset, sum, normalised O in fp16) in its own shared memory and, after a
// cluster barrier, CTA r merges the rows r, r + splits, ... of all partials through distributed shared memory
// in split order (deterministic) and writes the output.  More than 8 splits fall back to a global workspace
// and the separate combine kernel.
// The launch carries the programmatic-dependent-launch attribute: the prologue (barriers, TMEM allocation,
// descriptor prefetch) may overlap the tail of the previous kernel on the stream; nothing is read from or
// written to global memory before griddepcontrol.wait.
// Every mbarrier wait is bounded (200 ms): on expiry the CTA flags S4C_SEQ_TIMEOUT in status[b], stops
// waiting for anything else, still takes part in the cluster barriers, frees its TMEM and returns.
#include <cuda.h>
#include <cuda_fp16.h>
#include <math.h>

#include "s4c_common.cuh"
#include "tree_attention.cuh"

namespace s4c {

constexpr int kBM = 128;  // query rows per row tile (TMEM lanes)
constexpr int kBN = 64;   // cache slots per tile
constexpr int kMaxClusterSplits = 8;
constexpr long long kWaitLimitCycles = 400ll * 1000 * 1000;  // about 200 ms at the 1.965 GHz boost clock, longer below it
constexpr int kDrainBars = 4;  // one per issuer warp (at most three) and a spare
constexpr float kRescaleThreshold = 8.f;  // log2 units

template <int D, int NM, int TC = 1, int PUSH = 0>
struct TcCfg {
    static constexpr int kHalves = D / 64;           // 64-element (128-byte) swizzle atoms along d
    static constexpr int kQBytes = kBM * D * 2;      // one row tile of Q: 32 KB (d = 128)
    static constexpr int kTileBytes = kBN * D * 2;   // 16 KB: one K or V tile
    // PUSH == 1: 32 KB at the end of the tile area are set aside to receive the other splits' partials (see the kernel)
    // PUSH == 2: half an SM per CTA (two K/V stages at d = 128), so that two CTAs of a grid of several waves share an
    //            SM and one streams while the other starts or finishes
    static constexpr int kRecvBytes = PUSH == 1 ? 32768 : 0;
    static constexpr int kCtasPerSm = PUSH == 2 ? 2 : 1;
    static constexpr int kStages =
        PUSH == 2 ? (D == 128 ? 2 : 4) : (D == 128 ? (NM == 1 ? 6 : 5) : 8) - kRecvBytes / (2 * kTileBytes);
    static constexpr int kSmemData = NM * kQBytes + 2 * kStages * kTileBytes + kRecvBytes;
    // TMEM score buffers per row tile: two per softmax group; four where a single group leaves the columns free, so
    // that a product S = Q K^T need not wait for the P V product two tiles back
    static constexpr int kScoreBufs = (NM == 1 && TC == 1 && PUSH != 2) ? 4 : 2 * TC;
    static constexpr int kNumBars = 1 + 4 * kStages + (3 * kScoreBufs + TC) * NM + kDrainBars;
    // TMA warp, a QK issuer warp per row tile, one PV issuer warp.  (Two row tiles: 4 + 8 = 12 warps, three per scheduler,
    // so that a thread may hold 168 registers; a 13th warp would cap every thread at 128 and spill the softmax loop.)
    static constexpr int kRoleWarps = 2 + NM;
    static constexpr int kThreads = 32 * kRoleWarps + 128 * NM * TC;  // ... and four softmax warps per row tile (and turn)
    // A partial is parked, and travels between the CTAs of a cluster, as one exchange row: the normalised output row in fp16 (2^-11
    // relative, an eighth of the bf16 rounding of the result), then (offset, sum) in fp32, padded to 16 bytes so that
    // rows 2D + 16 bytes apart spread over the banks.  Half the bytes of fp32 rows on the slow path between SMs.
    static constexpr int kXRowBytes = 2 * D + 16;
    static constexpr int kXBytes = NM * TC * kBM * kXRowBytes;
    static constexpr int kSmemBytes = 1024 /*alignment slack*/ + kSmemData + 1024 /*barriers, flags, parent[]*/;
    static constexpr int kTmemCols = NM * kScoreBufs * kBN + NM * TC * D <= 256 ? 256 : 512;
    static_assert(kNumBars * 8 <= 480, "barrier area");
    static_assert(PUSH == 2 || 2 * kXBytes <= kSmemData, "parked partials reuse the tile buffers (half-SM CTAs never merge)");
    static_assert(kSmemBytes <= 232448, "shared memory per CTA");
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
// Bounded wait: true once the phase has completed, false when the wait was given up.  `dead` (shared memory) is set by
// the first wait of the CTA that runs out of time; every later wait then gives up at once.  A role that gets `false`
// leaves its loop without issuing anything further (no copy, no product, no tensor-memory store).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* dead, long long limit) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*dead) return false;
        if (clock64() - t0 > limit) {
            *dead = 1;
            return false;
        }
    }
}
// Whole-warp wait: lane 0 polls the barrier, the other lanes pick the result up at the warp barrier (one poller
// per warp instead of 32 keeps the shared-memory barrier unit free for the arrivals).  Whether the wait was given up
// shows in `dead`, which the caller reads where a warp-uniform answer costs nothing.
__device__ __forceinline__ void mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* dead, long long limit) {
    if ((threadIdx.x & 31) == 0) mbar_wait(bar, parity, dead, limit);
    __syncwarp();
}
// Wait for something this CTA itself set in motion (a bulk copy, a committed product) on the way out of a CTA that has
// given up: bounded like every wait, but not cut short by `dead`, so that nothing is still in flight into shared or
// tensor memory when the CTA frees them.
__device__ __forceinline__ void mbar_drain(uint32_t bar, uint32_t parity, long long limit) {
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity))
        if (clock64() - t0 > limit) return;
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
        "l"(map), "r"(bar), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(dst),
        "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
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
// Same product with the A operand in tensor memory: 128 lanes (rows) x 8 columns, each 32-bit cell two bf16 (the
// lower K index in the lower half).
__device__ __forceinline__ void tc_mma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
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
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
// N consecutive 32-bit columns of this thread's TMEM lane (N in {16, 32, 64}); the caller waits for the load.
template <int N>
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, uint32_t (&r)[N]) {
    static_assert(N == 16 || N == 32 || N == 64, "column count");
    if constexpr (N == 16) {
        tmem_ld16(taddr, r);
    } else if constexpr (N == 32) {
        tmem_ld32(taddr, r);
    } else {
        tmem_ld32(taddr, *reinterpret_cast<uint32_t(*)[32]>(&r[0]));
        tmem_ld32(taddr + 32, *reinterpret_cast<uint32_t(*)[32]>(&r[32]));
    }
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
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(taddr), "r"(r[0]),
                 "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}
// N consecutive 32-bit columns of this thread's TMEM lane (N in {8, 16, 32}); the caller waits for the store.
template <int N>
__device__ __forceinline__ void tmem_st_cols(uint32_t taddr, const uint32_t (&r)[N]) {
    static_assert(N == 8 || N == 16 || N == 32, "column count");
    if constexpr (N == 8) {
        tmem_st8(taddr, r);
    } else if constexpr (N == 16) {
        tmem_st16(taddr, r);
    } else {
        tmem_st32(taddr, r);
    }
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void st_cluster_f4(uint32_t addr, float a, float b, float c, float d) {
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ void st_cluster_f2(uint32_t addr, float a, float b) {
    asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(addr), "f"(a), "f"(b) : "memory");
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void st_cluster_u4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ uint2 ld_cluster_u2(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared::cluster.v2.b32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t ld_cluster_u1(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared::cluster.b32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
// Two floats to fp16 (a in the low half), saturating at the largest finite value: a normalised output row is a convex
// combination of V rows, so only V entries beyond +-65504 can reach the limit; they are clamped there rather than turned
// into infinities (which a zero weight would turn into NaN).
__device__ __forceinline__ uint32_t pack_half2(float a, float b) {
    uint32_t r;
    asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(b), "f"(a));
    return r;
}
__device__ __forceinline__ float2 unpack_half2(uint32_t v) { return __half22float2(*reinterpret_cast<const __half2*>(&v)); }
__device__ __forceinline__ float2 ld_cluster_f2(uint32_t addr) {
    float2 v;
    asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
}
// ---- packed pairs of floats (one instruction, two lanes of the FP32 pipe) and the three-input maximum
__device__ __forceinline__ uint64_t f2_pack(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f2_unpack(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t f2_sub(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// 2^x for a pair on the FP32 pipe instead of the special-function unit: x is split into its nearest integer n (adding
// 1.5 * 2^23 leaves n in the low mantissa bits) and f = x - n in [-1/2, 1/2]; a cubic (minimax, relative error 7.5e-5 --
// the result is rounded to bf16, 3.9e-3, right after) gives 2^f and n goes into the exponent.
__device__ __forceinline__ void exp2_pair_fma(uint64_t x2, float& p0, float& p1) {
    float x0, x1;
    f2_unpack(x2, x0, x1);
    x0 = fmaxf(x0, -126.f), x1 = fmaxf(x1, -126.f);  // masked columns arrive as -inf
    const uint64_t x = f2_pack(x0, x1);
    const uint64_t magic = f2_pack(12582912.f, 12582912.f);
    const uint64_t xr = f2_add(x, magic);
    const uint64_t f = f2_sub(x, f2_sub(xr, magic));
    uint64_t p = f2_fma(f2_pack(0x1.c3f760p-5f, 0x1.c3f760p-5f), f, f2_pack(0x1.f0de1ap-3f, 0x1.f0de1ap-3f));
    p = f2_fma(p, f, f2_pack(0x1.62f31ap-1f, 0x1.62f31ap-1f));
    p = f2_fma(p, f, f2_pack(0x1.fff692p-1f, 0x1.fff692p-1f));
    float r0, r1, n0, n1;
    f2_unpack(p, r0, r1);
    f2_unpack(xr, n0, n1);
    p0 = __uint_as_float(__float_as_uint(r0) + (__float_as_uint(n0) << 23));
    p1 = __uint_as_float(__float_as_uint(r1) + (__float_as_uint(n1) << 23));
}
__device__ __forceinline__ float max3f(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ void named_bar_sync(int id, int count) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

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

enum TcMode { kModeDirect = 0, kModeCluster = 1, kModeWorkspace = 2 };

struct TcParams {
    const int32_t* cache_len;
    const int32_t* parent;
    const int32_t* n_nodes;
    __nv_bfloat16* out;
    float* ws;
    int32_t* status;
    int T, Hq, Hkv, C, m_groups, splits, mode, q_box_rows;
    float scale_log2;
    long long wait_limit;  // clock cycles a wait may take (kWaitLimitCycles; the self-test passes a short one)
    int withhold_tile;     // -1; the self-test names one tile of every CTA that the producer does not request
    // paged caches (block_table == nullptr: one contiguous cache of C slots per sequence and KV head)
    const int32_t* block_table;  // [B, max_blocks]: page of logical block i of sequence b
    int max_blocks, page_tiles, n_pages;  // page_tiles = page size / 64 slots
    int out_rows;  // 0: out is [B,Hq,T,d]; 1: [B,T,Hq,d] -- rows (b, t) of width Hq*d, as the output projection reads them
};

// element offset of the output row of packed query row gr (= g * T + t, g the head within the KV head's group)
template <int ROWS>
__device__ __forceinline__ size_t out_row_offset(const TcParams& prm, int b, int first_head, int gr, int T, int D) {
    if (!ROWS) return ((size_t)(b * prm.Hq + first_head) * T + gr) * D;
    const int g = gr / T, t = gr - g * T;
    return (((size_t)b * T + t) * prm.Hq + first_head + g) * D;
}

// Tile range of a split: tiles are dealt out as evenly as whole tiles allow, the odd ones to the FIRST splits -- the last
// split holds the tree's own tiles, which cost more than a tile of the prefix (they are masked), and every split of a
// cluster waits for the slowest.
__device__ __forceinline__ void split_range(int n_tiles, int splits, int split, int& t0, int& t1) {
    // (at most 2^25 tiles and 64 splits: the products fit 32 bits, and a 32-bit division is a fraction of a 64-bit one)
    t0 = (int)(((uint32_t)n_tiles * (uint32_t)split + (uint32_t)splits - 1u) / (uint32_t)splits);
    t1 = (int)(((uint32_t)n_tiles * (uint32_t)(split + 1) + (uint32_t)splits - 1u) / (uint32_t)splits);
}

// REP > 1 (one row tile, G*T <= 128 / REP rows): the query rows are laid into the 128 MMA rows REP times
// (copy c at rows c*128/REP...), every copy sees the same scores and owns the columns [c*64/REP, (c+1)*64/REP)
// of each tile: its own running offset and sum, its own slice of P (the rest of its P rows stays zero), its
// own accumulator rows.  The copies are merged like splits.  This spreads the exponentials of a small tree
// over all four softmax warps instead of leaving them to one.
// TC == 2 (one row tile of 65..128 rows, no row copies): two softmax groups take turns, group c owning the tiles
// j = c, c+2, ... with score buffer c and an accumulator of its own -- a full 128-row tile keeps one softmax group
// busy for longer than a tile takes to arrive, two groups do not.  The two accumulators merge like splits.
// PUSH (one row tile, no turns, few rows): instead of parking partials for the peers to fetch, every CTA stores its
// (copy-merged) rows into a receive area of the row's owner that is used for nothing else, so no barrier has to say
// "my tile buffers are dead" first; after one cluster barrier the owner merges from its own shared memory and leaves.
template <int D, int NM, int REP, int TC, int PUSH, int ROWS = 0 /* 1: out is [B,T,Hq,d]; a variant of its own, so that the [B,Hq,T,d] kernels stay as they are */>
__global__ void __launch_bounds__(TcCfg<D, NM, TC, PUSH>::kThreads, TcCfg<D, NM, TC, PUSH>::kCtasPerSm)
tree_attention_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                         const __grid_constant__ CUtensorMap map_v, const TcParams prm) {
    static_assert(NM == 1 || REP == 1, "row copies only with a single row tile");
    static_assert(TC == 1 || (NM == 1 && REP == 1), "turns only with a single row tile and no row copies");
    static_assert(PUSH == 0 || (NM == 1 && TC == 1), "pushed partials and half-SM CTAs only with a single row tile and no turns");
    static_assert(PUSH != 1 || REP > 1, "partials are pushed by the threads that merged the row copies");
    using Cfg = TcCfg<D, NM, TC, PUSH>;
    constexpr int S = Cfg::kStages;
    constexpr int NH = Cfg::kHalves;
    constexpr int XS = Cfg::kXRowBytes;
    constexpr int RB = kBM / REP;  // rows per copy
    constexpr int CW = kBN / REP;  // columns of a tile per copy
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // 128B swizzle atoms need 1024-byte alignment
    unsigned char* base_ptr = smem_raw + (base - raw);
    const uint32_t sQ = base;
    const uint32_t sK = sQ + NM * Cfg::kQBytes;
    const uint32_t sV = sK + S * Cfg::kTileBytes;
    unsigned char* tail = base_ptr + Cfg::kSmemData;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 480);
    volatile int* dead = reinterpret_cast<volatile int*>(tail + 484);
    int* bad_s = reinterpret_cast<int*>(tail + 488);  // S4C_SEQ_* flags found by the softmax warps (malformed tree)
    int* issued_s = reinterpret_cast<int*>(tail + 492);  // tiles the producer has requested
    int32_t* par_s = reinterpret_cast<int32_t*>(tail + 512);  // S4C_MAX_T * 4 = 512 bytes

    const uint32_t bar0 = smem_u32(bars);
    auto BAR = [&](int i) { return bar0 + 8u * i; };
    // barrier indices; the per-row-tile ones take (tile t, buffer i)
    constexpr int Q_FULL = 0, K_FULL = 1, K_EMPTY = 1 + S, V_FULL = 1 + 2 * S, V_EMPTY = 1 + 3 * S, PER_TILE = 1 + 4 * S;
    constexpr int NB = Cfg::kScoreBufs, PT = 3 * NB + TC;  // score buffers and barriers per row tile; tile j uses buffer j % NB
    constexpr int DRAIN = PER_TILE + PT * NM;               // one per issuer warp: its products are complete (used when giving up)
    const long long limit = prm.wait_limit;
    auto S_FULL = [&](int t, int i) { return BAR(PER_TILE + PT * t + i); };
    auto S_EMPTY = [&](int t, int i) { return BAR(PER_TILE + PT * t + NB + i); };
    auto P_FULL = [&](int t, int i) { return BAR(PER_TILE + PT * t + 2 * NB + i); };
    auto PV_DONE = [&](int t, int c) { return BAR(PER_TILE + PT * t + 3 * NB + c); };  // c: the softmax group whose tile it was

    const int split = blockIdx.x, splits = prm.splits;
    const int mg = blockIdx.y % prm.m_groups, hk = blockIdx.y / prm.m_groups, b = blockIdx.z;
    const int T = prm.T, G = prm.Hq / prm.Hkv, R = G * T;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int mt0 = mg * NM;  // first row tile of this CTA
    auto rows_in = [&](int t) {  // valid query rows of row tile t of this CTA (per copy when REP > 1)
        const int r = R - (mt0 + t) * kBM;
        return r < 0 ? 0 : (r > kBM ? kBM : r);
    };
    auto active_threads = [&](int t) {  // softmax threads of row tile t whose warp owns at least one valid row
        return REP > 1 ? kBM : 32 * ((rows_in(t) + 31) / 32);
    };
    int nm_act = 0;  // row tiles with at least one row (they are the first ones)
#pragma unroll
    for (int t = 0; t < NM; ++t) nm_act += rows_in(t) > 0 ? 1 : 0;

    // ---- prologue that touches no global memory: barriers (one per lane of warp 0), TMEM, descriptor prefetch
    if (warp == 0) {
        for (int i = lane; i < Cfg::kNumBars; i += 32) {
            uint32_t count = 1;  // but: P_FULL takes one arrival per active softmax warp, the EMPTY barriers of
                                 // the ring one commit per active row tile (each has issuer threads of its own)
            if ((i >= K_EMPTY && i < K_EMPTY + S) || (i >= V_EMPTY && i < V_EMPTY + S)) count = (uint32_t)nm_act;
            if (i >= PER_TILE && i < DRAIN) {
                const int t = (i - PER_TILE) / PT, k = (i - PER_TILE) % PT;
                const uint32_t active = (uint32_t)active_threads(t) / 32u;
                if (k >= 2 * NB && k < 3 * NB && active) count = active;
            }
            mbar_init(BAR(i), count);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (lane == 0) {
            tma_prefetch_desc(&map_q), tma_prefetch_desc(&map_k), tma_prefetch_desc(&map_v);
            *dead = 0;
            *bad_s = 0;
            *issued_s = 0;
        }
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), Cfg::kTmemCols);
    tc_fence_before();
    __syncthreads();  // the only CTA-wide barrier before the results: from here on the roles run on mbarriers alone
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    auto TM_S = [&](int t, int i) { return tmem + (uint32_t)((t * NB + i) * kBN); };
    auto TM_O = [&](int t, int c) { return tmem + (uint32_t)(NM * NB * kBN + (t * TC + c) * D); };

    griddep_wait();  // everything below may depend on the previous kernel of the stream

    const int n = prm.n_nodes ? prm.n_nodes[b] : T;
    const int L = prm.cache_len[b];
    int flags = (n < 1 || n > T) ? S4C_SEQ_BAD_PARENT : 0;
    if (L < 0 || (long long)L + (n > 0 ? n : 0) > (long long)prm.C) flags |= S4C_SEQ_CAPACITY;
    const int Ltot = L + n;
    int t0 = 0, t1 = 0;
    if (!flags) split_range((Ltot + kBN - 1) / kBN, splits, split, t0, t1);
    const int nt = t1 - t0;  // 0 when the lengths are unusable: nothing is loaded, issued or stored then
    griddep_launch_dependents();

    const int q_row0 = (b * prm.Hq + hk * G) * T + mt0 * kBM;  // row of the [B*Hq*T, d] view of q
    const int kv_row0 = (b * prm.Hkv + hk) * prm.C;            // row of the [B*Hkv*C, d] view of the caches
    const uint32_t q_bytes = (uint32_t)prm.q_box_rows * 128u * NH;
    // Paged caches [n_pages, Hkv, page, d]: tile g of the sequence lies in the page its block table names; a page holds
    // whole tiles.  A page number outside the pool is flagged and replaced by page 0 (the copy stays inside the pool).
    auto fetch_page = [&](int g) -> int { return __ldg(prm.block_table + (size_t)b * prm.max_blocks + g / prm.page_tiles); };
    auto check_page = [&](int page) -> int {  // (apart from the fetch, so that the fetch's latency can pass behind other work)
        if ((unsigned)page >= (unsigned)prm.n_pages) {
            atomicOr(bad_s, S4C_SEQ_BAD_PAGE);
            page = 0;
        }
        return page;
    };
    auto lookup_page = [&](int g) -> int { return check_page(fetch_page(g)); };
    auto paged_row = [&](int g, int page) { return ((page * prm.Hkv + hk) * prm.page_tiles + g % prm.page_tiles) * kBN; };
    const bool paged = prm.block_table != nullptr;

    if (warp == 0) {
        // ================= TMA producer =================
        auto load_tile = [&](int j, int row) -> bool {  // false: a wait was given up, nothing further is requested
            const int s = j % S, it = j / S;
            if (j == prm.withhold_tile) return true;  // (self-test only: this tile never arrives)
            if (!mbar_wait(BAR(K_EMPTY + s), (it & 1) ^ 1, dead, limit)) return false;
            mbar_expect_tx(BAR(K_FULL + s), Cfg::kTileBytes);
            if (NH == 2) {  // one request per tile: the map's third dimension is the 64-column half
                tma_load_3d(sK + s * Cfg::kTileBytes, &map_k, BAR(K_FULL + s), 0, row, 0);
            } else {
                tma_load_2d(sK + s * Cfg::kTileBytes, &map_k, BAR(K_FULL + s), 0, row);
            }
            if (!mbar_wait(BAR(V_EMPTY + s), (it & 1) ^ 1, dead, limit)) {
                mbar_drain(BAR(K_FULL + s), it & 1, limit);  // the K half of this tile is on its way: see it in
                return false;
            }
            mbar_expect_tx(BAR(V_FULL + s), Cfg::kTileBytes);
            if (NH == 2) {
                tma_load_3d(sV + s * Cfg::kTileBytes, &map_v, BAR(V_FULL + s), 0, row, 0);
            } else {
                tma_load_2d(sV + s * Cfg::kTileBytes, &map_v, BAR(V_FULL + s), 0, row);
            }
            return true;
        };
        if (nt > 0) {
            // Q first (the requests are served in order, and the first product needs it): one request per lane -- a row
            // copy or row tile, and a 64-column half -- all at once; one thread needs about 50 ns per request
            if (lane == 0) mbar_expect_tx(BAR(Q_FULL), q_bytes * (REP > 1 ? REP : nm_act));
            if (REP > 1) {
                if (lane < REP * NH)  // the same rows once per copy, RB rows (whole swizzle atoms) apart
                    tma_load_2d(sQ + (lane % NH) * (kBM * 128) + (lane / NH) * (RB * 128), &map_q, BAR(Q_FULL), (lane % NH) * 64, q_row0);
            } else if (lane < nm_act * NH) {
                tma_load_2d(sQ + (lane / NH) * Cfg::kQBytes + (lane % NH) * (kBM * 128), &map_q, BAR(Q_FULL), (lane % NH) * 64,
                            q_row0 + (lane / NH) * kBM);
            }
            __syncwarp();
            // then the first pass of the ring, every ring slot still free: again one request per lane
            if (lane < 2 * S && (lane >> 1) < nt && (lane >> 1) != prm.withhold_tile) {
                // K and V of a tile on neighbouring lanes: the requests go out as K0 V0 K1 V1 ..., so that the first
                // product with V does not wait behind every K tile of the ring
                const int j = lane >> 1;
                const int row = paged ? paged_row(t0 + j, lookup_page(t0 + j)) : kv_row0 + (t0 + j) * kBN;
                const uint32_t full = BAR(((lane & 1) ? V_FULL : K_FULL) + j);
                const uint32_t dst = ((lane & 1) ? sV : sK) + j * Cfg::kTileBytes;
                const CUtensorMap* map = (lane & 1) ? &map_v : &map_k;
                mbar_expect_tx(full, Cfg::kTileBytes);
                if (NH == 2) {
                    tma_load_3d(dst, map, full, 0, row, 0);
                } else {
                    tma_load_2d(dst, map, full, 0, row);
                }
            }
            __syncwarp();
            if (lane == 0) {
                int issued = nt < S ? nt : S;
                // (paged: the page of the next tile is looked up before this tile's ring slot is waited for)
                int page_next = (paged && issued < nt) ? fetch_page(t0 + issued) : 0, page_after = 0;
                if (paged && issued + 1 < nt) page_after = fetch_page(t0 + issued + 1);
                for (; issued < nt; ++issued) {  // table entries are fetched two tiles ahead and looked at when needed
                    const int page = paged ? check_page(page_next) : 0;
                    page_next = page_after;
                    if (paged && issued + 2 < nt) page_after = fetch_page(t0 + issued + 2);
                    if (!load_tile(issued, paged ? paged_row(t0 + issued, page) : kv_row0 + (t0 + issued) * kBN)) break;
                }
                *issued_s = issued;  // tiles requested: what a CTA that gives up has to see in before it leaves
            }
            __syncwarp();
        }
    } else if (warp <= NM) {
        // ================= QK issuer of row tile t: S = Q K^T =================
        // (one issuing warp per product and row tile: a single thread spends more time issuing a tile's
        //  instructions and polling its barriers than the tile takes to arrive; the whole warp runs the loop so
        //  that the descriptor arithmetic is warp-uniform, one elected lane issues)
        const int t = warp - 1;
        if (nt > 0 && t < nm_act) {
            constexpr uint32_t idesc_qk = instr_desc_bf16(kBM, kBN, false);
            uint64_t a_desc[D / 16];  // the Q operand never moves: one descriptor per K step, made once
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk)  // 64-element halves along d, 32 bytes per K step inside a half
                a_desc[kk] = smem_desc_sw128(sQ + t * Cfg::kQBytes + (kk >> 2) * (kBM * 128) + (kk & 3) * 32, 16, 1024);
            // `ok` is this lane's own record: once one of its waits has been given up it never issues again.  (The lanes
            // poll on their own and need not agree at the moment of giving up; the elected lane acts on what it saw
            // itself, and every later wait of every lane ends at once.)
            bool ok = mbar_wait(BAR(Q_FULL), 0, dead, limit);
            for (int j = 0; j < nt; ++j) {
                const int s = j % S, it = j / S;
                ok &= mbar_wait(BAR(K_FULL + s), it & 1, dead, limit);
                const uint64_t k_desc = smem_desc_sw128(sK + s * Cfg::kTileBytes, 16, 1024);
                ok &= mbar_wait(S_EMPTY(t, j % NB), ((j / NB) & 1) ^ 1, dead, limit);
                tc_fence_after();
                if (elect_one() && ok) {
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk)  // the start-address field counts 16-byte units
                        tc_mma_bf16(TM_S(t, j % NB), a_desc[kk], k_desc + (uint64_t)(((kk >> 2) * (kBN * 128) + (kk & 3) * 32) >> 4),
                                    idesc_qk, kk > 0 ? 1u : 0u);
                    tc_commit(S_FULL(t, j % NB));
                    tc_commit(BAR(K_EMPTY + s));
                }
                __syncwarp();
            }
        }
    } else if (warp == NM + 1) {
        // ================= PV issuer: O += P V, for every row tile in turn =================
        // (the row tiles' softmax groups finish a tile one after the other, so one warp serves them in that order)
        if (nt > 0) {
            constexpr uint32_t idesc_pv = instr_desc_bf16(kBM, D, true);
            bool ok = true;  // this lane's own record, as in the QK issuer
            for (int j = 0; j < nt; ++j) {
                const int s = j % S, it = j / S;
                ok &= mbar_wait(BAR(V_FULL + s), it & 1, dead, limit);
                if ((t0 + j) * kBN + kBN > Ltot) {
                    // last, partial tile of the sequence: rows past the end may hold anything (even NaN); P is 0 there
                    // but 0 * NaN would poison O, so those V rows are cleared before the product reads them -- here, by
                    // the warp that waits for P anyway
                    const int first = Ltot - (t0 + j) * kBN;  // 1..63
                    unsigned char* vt = base_ptr + (sV - base) + s * Cfg::kTileBytes;
                    constexpr int CPR = 8 * NH;  // 16-byte chunks per slot: a lane keeps its chunk and walks down the slots
                    for (int r = first + lane / CPR; r < kBN; r += 32 / CPR)
                        *reinterpret_cast<uint4*>(vt + ((lane % CPR) >> 3) * (kBN * 128) + r * 128 + (lane & 7) * 16) = make_uint4(0, 0, 0, 0);
                    fence_async_smem();  // generic-proxy stores, read by the tensor core through the async proxy
                    __syncwarp();
                }
                // B = V [64 slots][d], MN-major: 16 slots (K step) = 2048 bytes; d halves kBN*128 bytes apart
                const uint64_t v_desc = smem_desc_sw128(sV + s * Cfg::kTileBytes, kBN * 128, 1024);
#pragma unroll
                for (int t = 0; t < NM; ++t) {
                    if (t >= nm_act) break;
                    ok &= mbar_wait(P_FULL(t, j % NB), (j / NB) & 1, dead, limit);
                    tc_fence_after();
                    if (elect_one() && ok) {
#pragma unroll
                        for (int kk = 0; kk < kBN / 16; ++kk)
                            // A = P in tensor memory, over the first 32 columns of the score buffer: 8 columns per K step
                            tc_mma_bf16_ts(TM_O(t, TC == 2 ? (j & 1) : 0), TM_S(t, j % NB) + kk * 8, v_desc + (uint64_t)((kk * 2048) >> 4),
                                           idesc_pv, (j >= TC || kk > 0) ? 1u : 0u);
                        tc_commit(PV_DONE(t, TC == 2 ? (j & 1) : 0));
                        tc_commit(S_EMPTY(t, j % NB));  // the score buffer (and the P inside it) may be overwritten
                        tc_commit(BAR(V_EMPTY + s));    // (one arrival per row tile)
                    }
                    __syncwarp();
                }
            }
        }
    } else {
        // ================= softmax / correction: one thread per MMA row =================
        // tree check first: softmax thread i looks at node i; a malformed tree still runs the pipeline (with empty
        // masks, so that no role waits for another) and only its outputs are withheld
        if (!flags) {
            const int i = threadIdx.x - 32 * Cfg::kRoleWarps;
            if (i < T) {
                const int p = prm.parent[(size_t)b * T + i];
                par_s[i] = p;
                if (i < n && ((i == 0 && p != -1) || (i > 0 && (p < 0 || p >= i)))) atomicOr(bad_s, S4C_SEQ_BAD_PARENT);
            }
        }
        named_bar_sync(1, NM * TC * 128);
        flags |= *bad_s;
        if (split == 0 && blockIdx.y == 0 && threadIdx.x == 32 * Cfg::kRoleWarps && prm.status) prm.status[b] = flags;
        const bool run = flags == 0;
        const int grp = (warp - Cfg::kRoleWarps) >> 2;  // this warp group: a row tile, or (TC == 2) a turn on the one row tile
        const int t = TC == 2 ? 0 : grp, tc = TC == 2 ? grp : 0;
        const int n_own = nt > tc ? (nt - tc + TC - 1) / TC : 0;  // tiles this group takes: tc, tc + TC, ...
        const int wq = warp & 3;        // TMEM lane quadrant this warp may access
        const int row = wq * 32 + lane;
        const int copy = row / RB, lr = row % RB;  // which copy of the rows, and the row within it
        const int rows_t = rows_in(t);
        const bool warp_active = REP > 1 || wq * 32 < rows_t;
        const bool row_ok = lr < rows_t;
        const int gr = (mt0 + t) * kBM + lr;
        const int node = gr % T;
        const int c0 = copy * CW;  // first tile column of this copy
        // the row's ancestor-or-self set as a 128-bit mask, straight from parent[] (checked above: the chain ends)
        uint64_t anc_lo = 0, anc_hi = 0;
        if (run && row_ok && node < n)
            for (int u = node, guard = 0; u >= 0 && guard <= T; u = par_s[u], ++guard) {
                if (u < 64)
                    anc_lo |= 1ull << u;
                else
                    anc_hi |= 1ull << (u - 64);
            }
        const uint32_t lane_off = (uint32_t)(wq * 32) << 16;
        float m = -1e30f, l = 0.f;  // m: offset in use (scaled, log2 units); never -inf so that exp2(-inf - m) = 0
        const float sc = prm.scale_log2;
        bool alive = true;  // false once this warp has seen a wait of the CTA given up

        if (warp_active)
            for (int j = tc; j < nt; j += TC) {
                const int kv0 = (t0 + j) * kBN;
                mbar_wait_warp(S_FULL(t, j % NB), (j / NB) & 1, dead, limit);
                tc_fence_after();
                float sv[CW];
                {
                    uint32_t sr[CW];
                    tmem_ld_cols<CW>(TM_S(t, j % NB) + lane_off + c0, sr);
                    const int gave_up = *dead;  // one word for the whole warp, read while the scores are on their way
                    tmem_wait_ld();
                    if (gave_up) {  // a wait of this CTA ran out: nothing further is computed or stored
                        alive = false;
                        break;
                    }
#pragma unroll
                    for (int c = 0; c < CW; ++c) sv[c] = __uint_as_float(sr[c]);
                }
                if (kv0 + kBN > L) {
                    // the tile touches tree slots or the tail: column c is visible iff it lies in the prefix or is the
                    // slot of a node on this row's root path
                    const int off = L - kv0;  // prefix columns of this tile (<= 0: none)
                    uint64_t vis;
                    if (off >= 0) {
                        vis = (anc_lo << off) | ((1ull << off) - 1ull);  // off < 64 here
                    } else {
                        const int sh = -off;  // first tree node of the tile
                        vis = sh < 64 ? ((anc_lo >> sh) | (anc_hi << (64 - sh))) : (sh < 128 ? (anc_hi >> (sh - 64)) : 0ull);
                    }
                    vis >>= c0;
                    const uint32_t v0 = (uint32_t)vis, v1 = (uint32_t)(vis >> 32);
#pragma unroll
                    for (int c = 0; c < CW; ++c) {
                        const bool on = (((c < 32 ? v0 : v1) >> (c & 31)) & 1u) != 0;
                        sv[c] = on ? sv[c] : -INFINITY;
                    }
                }
                float mx4[4] = {sv[0], sv[1], sv[2], sv[3]};  // four independent chains, two columns per instruction
#pragma unroll
                for (int c = 4; c < CW; c += 2) mx4[(c >> 1) & 3] = max3f(mx4[(c >> 1) & 3], sv[c], sv[c + 1]);
                const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * sc;  // sc > 0
                const bool grow = row_ok && mx > m + kRescaleThreshold;
                const float m_new = grow ? mx : m;
                const float alpha = grow ? exp2f(m - m_new) : 1.f;
                // exponentials and their sums in pairs.  With two row tiles, two softmax warps share each scheduler's
                // special-function unit (16 lanes per SM) and it is what a tile waits for: one pair in four goes through
                // the FP32 pipe instead.
                const uint64_t sc2 = f2_pack(sc, sc), nm2 = f2_pack(-m_new, -m_new);
                uint64_t ls2[2] = {f2_pack(0.f, 0.f), f2_pack(0.f, 0.f)};
                uint32_t pk[CW / 2];
#pragma unroll
                for (int c = 0; c < CW; c += 2) {
                    const uint64_t x2 = f2_fma(f2_pack(sv[c], sv[c + 1]), sc2, nm2);
                    float p0, p1;
                    if ((NM == 2) && ((c >> 1) & 3) == 3) {
                        exp2_pair_fma(x2, p0, p1);
                    } else {
                        float x0, x1;
                        f2_unpack(x2, x0, x1);
                        p0 = exp2f(x0), p1 = exp2f(x1);
                    }
                    ls2[(c >> 1) & 1] = f2_add(ls2[(c >> 1) & 1], f2_pack(p0, p1));
                    const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
                    pk[c >> 1] = *reinterpret_cast<const uint32_t*>(&h2);
                }
                {
                    float a0, a1, b0, b1;
                    f2_unpack(ls2[0], a0, a1);
                    f2_unpack(ls2[1], b0, b1);
                    l = l * alpha + ((a0 + a1) + (b0 + b1));
                }
                m = m_new;

                // O is rescaled (rarely) once this group's previous product, number i - 1 on its own barrier, is complete.
                // With two score buffers per group S_FULL of tile i already says that product i - 2 is complete, so the
                // barrier is at most one phase behind whenever it is looked at and the look can be left out when no row
                // of the warp moves its offset -- except on the group's last tile, so that the wait after the loop
                // finds it at most one phase behind as well.  (Four buffers: product i - 4 only; the wait stays.)
                const int i_own = (j - tc) / TC;
                const bool any_grow = __any_sync(0xffffffffu, grow);
                if (i_own > 0 && (NB != 2 * TC || any_grow || i_own == n_own - 1)) {
                    mbar_wait_warp(PV_DONE(t, tc), (i_own - 1) & 1, dead, limit);
                    tc_fence_after();
                    if (any_grow) {
#pragma unroll
                        for (int cc = 0; cc < D / 32; ++cc) {
                            uint32_t o[32];
                            tmem_ld_cols<32>(TM_O(t, tc) + lane_off + cc * 32, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
                            tmem_st32(TM_O(t, tc) + lane_off + cc * 32, o);
                        }
                        tmem_wait_st();
                    }
                }
                // P row -> tensor memory, packed two bf16 per column over the first 32 columns of this score buffer (the
                // scores were read above).  A copy owns CW/2 of these columns and clears the others: the product runs
                // over all 64 slots of every row.
                {
                    const uint32_t p_row = TM_S(t, j % NB) + lane_off;
                    tmem_st_cols<CW / 2>(p_row + c0 / 2, pk);
                    if (REP > 1) {
                        uint32_t zero[CW / 2];
#pragma unroll
                        for (int c = 0; c < CW / 2; ++c) zero[c] = 0u;
#pragma unroll
                        for (int k = 1; k < REP; ++k) tmem_st_cols<CW / 2>(p_row + ((copy + k) % REP) * (CW / 2), zero);
                    }
                    tmem_wait_st();
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(P_FULL(t, j % NB));
            }

        // ---- this split's (and copy's) result for the row: (m, l, unnormalised O)
        if (warp_active && n_own > 0) {
            mbar_wait_warp(PV_DONE(t, tc), (n_own - 1) & 1, dead, limit);
            tc_fence_after();
        }
        const bool node_valid = row_ok && node < n;
        if (prm.mode == kModeCluster) {
            // every MMA of the CTA has finished before any tile buffer is reused for the parked partials
            named_bar_sync(1, NM * TC * 128);
            // a warp that saw a wait of its CTA given up parks, merges and stores nothing (copies may still be landing in
            // the tile buffers); it keeps taking the barriers so that nobody waits for it
            if (warp_active && alive) {
                // the thread's row (of its copy, of its turn) is parked as an exchange row
                unsigned char* xo = base_ptr + (size_t)((t * TC + tc) * kBM + row) * XS;
                const float inv_l = (n_own > 0 && l > 0.f) ? 1.f / l : 0.f;
#pragma unroll
                for (int cc = 0; cc < D / 64; ++cc) {  // 64 columns per round trip to tensor memory
                    uint32_t o[64];
                    if (n_own > 0) {
                        tmem_ld_cols<64>(TM_O(t, tc) + lane_off + cc * 64, o);
                        tmem_wait_ld();
                    } else {
#pragma unroll
                        for (int c = 0; c < 64; ++c) o[c] = 0u;
                    }
#pragma unroll
                    for (int c = 0; c < 64; c += 8)
                        *reinterpret_cast<uint4*>(xo + (cc * 64 + c) * 2) =
                            make_uint4(pack_half2(__uint_as_float(o[c]) * inv_l, __uint_as_float(o[c + 1]) * inv_l),
                                       pack_half2(__uint_as_float(o[c + 2]) * inv_l, __uint_as_float(o[c + 3]) * inv_l),
                                       pack_half2(__uint_as_float(o[c + 4]) * inv_l, __uint_as_float(o[c + 5]) * inv_l),
                                       pack_half2(__uint_as_float(o[c + 6]) * inv_l, __uint_as_float(o[c + 7]) * inv_l));
                }
                *reinterpret_cast<float2*>(xo + 2 * D) = make_float2(m, inv_l > 0.f ? l : 0.f);
            }
            if (REP > 1) {
                // The copies of a row are merged here, inside the CTA, before the splits are merged across the
                // cluster: distributed shared memory is slow, so it should carry one partial per split and row, not
                // REP.  Thread (r, q) of the 128 merges columns [q D/REP, (q+1) D/REP) of row r from all copies, in
                // copy order (the same on every run).
                named_bar_sync(1, 128);
                constexpr int CPT = D / REP;  // columns per thread
                const int tid = (int)threadIdx.x - 32 * Cfg::kRoleWarps;
                const int r = tid % RB, col0 = (tid / RB) * CPT;
                const bool mine = r < rows_t && alive;
                float acc[CPT], M = -INFINITY, den = 0.f;
#pragma unroll
                for (int k = 0; k < CPT; ++k) acc[k] = 0.f;
                if (mine) {
                    float2 ml[REP];
#pragma unroll
                    for (int c = 0; c < REP; ++c) {
                        ml[c] = *reinterpret_cast<const float2*>(base_ptr + (size_t)(c * RB + r) * XS + 2 * D);
                        M = fmaxf(M, ml[c].x);
                    }
#pragma unroll
                    for (int c = 0; c < REP; ++c) {
                        const float w = exp2f(ml[c].x - M) * ml[c].y;  // the copy's share of the softmax sum
                        den += w;
                        const unsigned char* src = base_ptr + (size_t)(c * RB + r) * XS + col0 * 2;
#pragma unroll
                        for (int k = 0; k < CPT; k += 8) {
                            const uint4 v = *reinterpret_cast<const uint4*>(src + k * 2);
                            const float2 a0 = unpack_half2(v.x), a1 = unpack_half2(v.y), a2 = unpack_half2(v.z), a3 = unpack_half2(v.w);
                            acc[k] = fmaf(w, a0.x, acc[k]), acc[k + 1] = fmaf(w, a0.y, acc[k + 1]);
                            acc[k + 2] = fmaf(w, a1.x, acc[k + 2]), acc[k + 3] = fmaf(w, a1.y, acc[k + 3]);
                            acc[k + 4] = fmaf(w, a2.x, acc[k + 4]), acc[k + 5] = fmaf(w, a2.y, acc[k + 5]);
                            acc[k + 6] = fmaf(w, a3.x, acc[k + 6]), acc[k + 7] = fmaf(w, a3.y, acc[k + 7]);
                        }
                    }
                }
                // the merged partial becomes one exchange row, straight from the registers
                const float inv_den = den > 0.f ? 1.f / den : 0.f;
                uint32_t hx[CPT / 2];
#pragma unroll
                for (int k = 0; k < CPT; k += 2) hx[k >> 1] = pack_half2(acc[k] * inv_den, acc[k + 1] * inv_den);
                if (PUSH == 1) {
                    // ... stored to CTA r % splits, slot (r / splits) * splits + split of its receive area
                    if (mine && run) {
                        const uint32_t recv = base + (uint32_t)(Cfg::kQBytes + 2 * S * Cfg::kTileBytes);
                        const uint32_t dst = map_to_cta(recv + (uint32_t)(((r / splits) * splits + split) * XS), (uint32_t)(r % splits));
#pragma unroll
                        for (int k = 0; k < CPT / 2; k += 4)
                            st_cluster_u4(dst + (uint32_t)(col0 * 2 + k * 4), hx[k], hx[k + 1], hx[k + 2], hx[k + 3]);
                        if (col0 == 0) st_cluster_f2(dst + (uint32_t)(2 * D), M, den);
                    }
                } else if (mine) {
                    // ... left behind the parked copies, where the peers will fetch it
                    unsigned char* xo = base_ptr + Cfg::kXBytes + (size_t)r * XS;
#pragma unroll
                    for (int k = 0; k < CPT / 2; k += 4)
                        *reinterpret_cast<uint4*>(xo + col0 * 2 + k * 4) = make_uint4(hx[k], hx[k + 1], hx[k + 2], hx[k + 3]);
                    if (col0 == 0) *reinterpret_cast<float2*>(xo + 2 * D) = make_float2(M, den);
                }
            }
        } else if (warp_active && run && alive) {
            const bool direct = prm.mode == kModeDirect;  // REP == 1 then
            const size_t orow = (size_t)(b * prm.Hq + hk * G) * T + gr;  // row of the [B*Hq*T, d] view of out
            const float inv = (node_valid && l > 0.f) ? 1.f / l : 0.f;
            // workspace: every (split, row copy or turn) is one partial of the row
            float* wrow = prm.ws + (orow * (size_t)(splits * REP * TC) + (size_t)(split * REP * TC + (TC == 2 ? tc : copy))) * (D + 2);
#pragma unroll
            for (int cc = 0; cc < D / 32; ++cc) {
                uint32_t o[32];
                if (n_own > 0) {
                    tmem_ld_cols<32>(TM_O(t, tc) + lane_off + cc * 32, o);
                    tmem_wait_ld();
                } else {
#pragma unroll
                    for (int c = 0; c < 32; ++c) o[c] = 0u;
                }
                if (!row_ok) continue;
                if (direct) {
                    uint32_t packed[16];
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        const __nv_bfloat162 h2 =
                            __floats2bfloat162_rn(__uint_as_float(o[c]) * inv, __uint_as_float(o[c + 1]) * inv);
                        packed[c >> 1] = *reinterpret_cast<const uint32_t*>(&h2);
                    }
                    uint4* dst = reinterpret_cast<uint4*>(prm.out + out_row_offset<ROWS>(prm, b, hk * G, gr, T, D) + cc * 32);
#pragma unroll
                    for (int v = 0; v < 4; ++v)
                        dst[v] = make_uint4(packed[4 * v], packed[4 * v + 1], packed[4 * v + 2], packed[4 * v + 3]);
                } else {
                    float* w = wrow + cc * 32;
                    if (!node_valid) {
#pragma unroll
                        for (int c = 0; c < 32; ++c) o[c] = 0u;
                    }
#pragma unroll
                    for (int c = 0; c < 32; c += 2)
                        *reinterpret_cast<float2*>(w + c) = make_float2(__uint_as_float(o[c]), __uint_as_float(o[c + 1]));
                }
            }
            if (!direct && row_ok)
                *reinterpret_cast<float2*>(wrow + D) = make_float2(node_valid ? m : -INFINITY, node_valid ? l : 0.f);
        }
        tc_fence_before();
    }

    if (PUSH == 1 && prm.mode == kModeCluster) {
        // ---- every split's partial of this CTA's rows (rank, rank + splits, ...) has been stored into its receive area
        __syncwarp();
        cluster_sync_all();
        const bool run = (flags | *bad_s) == 0;
        const int gave_up = *dead;  // (a CTA that gave up stores nothing; only the stores wait for this word)
        const uint32_t rank = cluster_ctarank();
        const unsigned char* recv = base_ptr + Cfg::kQBytes + 2 * S * Cfg::kTileBytes;
        constexpr int EPL = D / 32;
        const int rows = rows_in(0);
        if (run)
            for (int k = warp; (int)rank + splits * k < rows; k += Cfg::kThreads / 32) {
                const int lr = (int)rank + splits * k;
                const unsigned char* prow = recv + (size_t)k * splits * XS;
                // every lane reads all (offset, sum) pairs itself (broadcast reads of this CTA's own shared memory):
                // no chain of shuffles between the barrier and the stores
                float M = -INFINITY;
                for (int i = 0; i < splits; ++i) M = fmaxf(M, *reinterpret_cast<const float*>(prow + (size_t)i * XS + 2 * D));
                float den = 0.f, num[4] = {0.f, 0.f, 0.f, 0.f};
                for (int i = 0; i < splits; ++i) {  // split order: the same on every run
                    const float2 ml = *reinterpret_cast<const float2*>(prow + (size_t)i * XS + 2 * D);
                    const float w = exp2f(ml.x - M) * ml.y;  // the partial's share of the softmax sum
                    den += w;
                    const unsigned char* src = prow + (size_t)i * XS + lane * (EPL * 2);
                    const float2 a = unpack_half2(*reinterpret_cast<const uint32_t*>(src));
                    num[0] = fmaf(w, a.x, num[0]), num[1] = fmaf(w, a.y, num[1]);
                    if (EPL == 4) {
                        const float2 c = unpack_half2(*reinterpret_cast<const uint32_t*>(src + 4));
                        num[2] = fmaf(w, c.x, num[2]), num[3] = fmaf(w, c.y, num[3]);
                    }
                }
                const int gr = mt0 * kBM + lr;
                const float inv = ((gr % T) < n && den > 0.f) ? 1.f / den : 0.f;
                __nv_bfloat16* dst = prm.out + out_row_offset<ROWS>(prm, b, hk * G, gr, T, D) + lane * EPL;
                const __nv_bfloat162 h0 = __floats2bfloat162_rn(num[0] * inv, num[1] * inv);
                if (gave_up) break;
                if (EPL == 4) {
                    const __nv_bfloat162 h1 = __floats2bfloat162_rn(num[2] * inv, num[3] * inv);
                    *reinterpret_cast<uint2*>(dst) =
                        make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1));
                } else {
                    *reinterpret_cast<uint32_t*>(dst) = *reinterpret_cast<const uint32_t*>(&h0);
                }
            }
        __syncthreads();  // warp 1 frees the tensor memory below: every warp is done
    } else if (prm.mode == kModeCluster) {
        // ---- merge the splits (and turns) through distributed shared memory: this CTA owns the output rows
        //      rank, rank + splits, ... of every row tile.  One warp per row, two rows at a time: lane i fetches
        //      (offset, sum) of partial i, every lane its 4 (d = 64: 2) output columns of up to 8 partials of both rows,
        //      all requests in flight before the first use -- a remote read takes about a microsecond
        __syncwarp();
        cluster_sync_all();
        // the same in every CTA of the cluster: it depends on the sequence only
        const bool run = (flags | *bad_s) == 0;
        const int gave_up = *dead;  // a CTA that gave up a wait stores nothing; only the stores wait for this word
        const uint32_t rank = cluster_ctarank();
        // row copies were merged inside their CTA (one exchange row per row, behind the parked copies); turns are
        // merged here with the splits
        const uint32_t part = base + (uint32_t)(REP > 1 ? Cfg::kXBytes : 0);
        constexpr int EPL = D / 32;  // output elements per lane
        constexpr int NC = TC;       // partials per split
        constexpr int U = 2;         // output rows in flight per warp
        const int np = splits * NC;  // partials per output row (<= 16)
        // exchange row of partial i of output row (t, lr): i / NC is the split, i % NC the turn
        auto part_addr = [&](int t, int lr, int i) {
            return map_to_cta(part + (uint32_t)(((t * TC + i % NC) * kBM + lr) * XS), (uint32_t)(i / NC));
        };
        const int stride = splits * (Cfg::kThreads / 32);
        if (run)
            for (int idx0 = (int)rank + splits * warp; idx0 < NM * RB; idx0 += U * stride) {
                int tt[U], lr[U];
                bool ok[U];
                float2 ml[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int idx = idx0 + u * stride;
                    tt[u] = idx / RB, lr[u] = idx % RB;
                    ok[u] = idx < NM * RB && lr[u] < rows_in(tt[u]);
                    ml[u] = make_float2(-INFINITY, 0.f);
                    if (ok[u] && lane < np) ml[u] = ld_cluster_f2(part_addr(tt[u], lr[u], lane) + (uint32_t)(2 * D));
                }
                float num[U][4], den[U], w_mine[U];
#pragma unroll
                for (int u = 0; u < U; ++u) num[u][0] = num[u][1] = num[u][2] = num[u][3] = 0.f, den[u] = 0.f;
                for (int i0 = 0; i0 < np; i0 += 8) {
                    uint2 h[U][8];
#pragma unroll
                    for (int u = 0; u < U; ++u)
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            h[u][k] = make_uint2(0u, 0u);
                            if (ok[u] && i0 + k < np) {
                                const uint32_t a = part_addr(tt[u], lr[u], i0 + k) + (uint32_t)(lane * EPL * 2);
                                if (EPL == 4) {
                                    h[u][k] = ld_cluster_u2(a);
                                } else {
                                    h[u][k].x = ld_cluster_u1(a);
                                }
                            }
                        }
                    if (i0 == 0) {
#pragma unroll
                        for (int u = 0; u < U; ++u) {
                            float M = -INFINITY;  // independent shuffles, not a butterfly: they overlap
                            for (int i = 0; i < np; ++i) M = fmaxf(M, __shfl_sync(0xffffffffu, ml[u].x, i));
                            w_mine[u] = lane < np ? exp2f(ml[u].x - M) * ml[u].y : 0.f;  // the partial's share of the sum
                        }
                    }
#pragma unroll
                    for (int u = 0; u < U; ++u)
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            const float w = __shfl_sync(0xffffffffu, w_mine[u], (i0 + k) & 31);  // 0 past the last partial
                            den[u] += w;  // partial order: the same on every run
                            const float2 a = unpack_half2(h[u][k].x), c = unpack_half2(h[u][k].y);
                            num[u][0] = fmaf(w, a.x, num[u][0]), num[u][1] = fmaf(w, a.y, num[u][1]);
                            num[u][2] = fmaf(w, c.x, num[u][2]), num[u][3] = fmaf(w, c.y, num[u][3]);
                        }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (!ok[u] || gave_up) continue;
                    const int gr = (mt0 + tt[u]) * kBM + lr[u];
                    const float inv = ((gr % T) < n && den[u] > 0.f) ? 1.f / den[u] : 0.f;
                    __nv_bfloat16* dst = prm.out + out_row_offset<ROWS>(prm, b, hk * G, gr, T, D) + lane * EPL;
                    const __nv_bfloat162 h0 = __floats2bfloat162_rn(num[u][0] * inv, num[u][1] * inv);
                    if (EPL == 4) {
                        const __nv_bfloat162 h1 = __floats2bfloat162_rn(num[u][2] * inv, num[u][3] * inv);
                        *reinterpret_cast<uint2*>(dst) =
                            make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1));
                    } else {
                        *reinterpret_cast<uint32_t*>(dst) = *reinterpret_cast<const uint32_t*>(&h0);
                    }
                }
            }
        __syncwarp();
        cluster_sync_all();  // nobody leaves while a peer may still read its shared memory
    } else {
        __syncthreads();
    }
    if (threadIdx.x == 0 && (*bad_s & S4C_SEQ_BAD_PAGE) && prm.status) atomicOr(prm.status + b, S4C_SEQ_BAD_PAGE);
    if (*dead) {  // read behind a CTA-wide barrier: the same in every thread
        // A wait was given up.  Before shared and tensor memory are handed back, everything this CTA set in motion is
        // seen to completion (bounded like every wait): a bulk copy that lands after the CTA has left would land in its
        // successor on the SM, a product that still runs would write tensor memory that is no longer this CTA's.
        if (warp == 0 && lane == 0 && nt > 0) {
            const int issued = *issued_s;
            mbar_drain(BAR(Q_FULL), 0, limit);
            for (int j = issued > S ? issued - S : 0; j < issued; ++j)
                if (j != prm.withhold_tile)
                    mbar_drain(BAR(K_FULL + j % S), (j / S) & 1, limit), mbar_drain(BAR(V_FULL + j % S), (j / S) & 1, limit);
        }
        if (warp >= 1 && warp <= NM + 1) {  // the issuer warps: a commit covers the products its own thread issued
            if (elect_one()) tc_commit(BAR(DRAIN + warp - 1));
            __syncwarp();
            mbar_drain(BAR(DRAIN + warp - 1), 0, limit);
        }
        __syncthreads();
        if (threadIdx.x == 0 && prm.status) atomicOr(prm.status + b, S4C_SEQ_TIMEOUT);
    }
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

// The same [rows, 128] matrix seen as [2 halves][rows][64 columns]: one box of 64 columns x box_rows x 2 halves lands in
// shared memory half by half, each half a stack of 128-byte rows -- the layout the K-major / MN-major operand
// descriptors of the kernel expect -- so a whole K or V tile takes one request.
static bool make_map_halves(CUtensorMap* map, const void* ptr, uint64_t rows, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {64, (cuuint64_t)rows, 2};
    const cuuint64_t strides[2] = {256, 128};  // bytes: next row, next half
    const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 2};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool tc_supported(int T, int Hq, int Hkv, int d, s4c_dtype dt) { return dt == S4C_BF16 && (d == 128 || d == 64); }

static int tc_m_tiles(int T, int Hq, int Hkv) { return ceil_div((Hq / Hkv) * T, kBM); }
// Row tiles per CTA.  Two row tiles on one K/V stream read K/V once for all rows of a KV head.  A grid of few (sequence,
// KV head) pairs cannot fill the GPU that way with the splits a cluster allows; one row tile per CTA then doubles the
// CTAs, the second read of a K/V tile being served by L2 (measured at 256 rows: 1 sequence x 8 KV heads, L=1024: 21.8 ->
// 9.2 us; 2 x 8, L=4096: 33.8 -> 18.6 us; 512 rows, 1 x 8, L=8192: 48 -> 27 us).  Only a single sequence of exactly two row
// tiles keeps both on one CTA beyond ~6k tokens (38 against 52 us at 16k).
static int tc_nm(int B, int T, int Hq, int Hkv, int C) {
    const int mt = tc_m_tiles(T, Hq, Hkv);
    if (mt <= 1) return 1;
    const int pairs = B * Hkv;
    if (pairs * ceil_div(mt, 2) * kMaxClusterSplits >= 148) return 2;
    return (mt == 2 && pairs < 12 && ceil_div(C, kBN) > 96) ? 2 : 1;
}
static int tc_m_groups(int B, int T, int Hq, int Hkv, int C) {
    return ceil_div(tc_m_tiles(T, Hq, Hkv), tc_nm(B, T, Hq, Hkv, C));
}

// Number of splits of the cache: the count that minimises waves x (fixed cost of a CTA + its tiles), with a small
// charge per extra split for the merge; a split has at least two tiles.  The fixed cost (set-up, first tile's latency,
// merge, measured at 5-6 us) is worth about ten tiles.  Up to 8 splits merge inside a cluster; a grid too small to
// fill the GPU even with 8 stays with 8 all the same -- the second launch and the fp32 partials in global memory of the
// wide path cost more than the idle SMs (8 heads, L=2048: 26.7 -> 8.2 us; 4 heads, L=8192: 38.6 -> 12.7 us) -- except for
// two row tiles per CTA on a very long cache, which go wider and merge through the workspace (53 against 66 us at 32k).
// CTAs that run at the same time when launched as clusters of s: asked of the device once (clusters do not straddle
// GPCs, and how many SMs a GPC offers to a cluster differs between GPCs and parts: clusters of 6 and of 8 measured two
// waves where 18 or 16 SMs per GPC would have held them in one).  Without a device the model of 16 SMs per GPC answers.
static int tc_resident_ctas(int s) {
    if (s == 1) return 148;
    static int table[64][kMaxClusterSplits + 1] = {};
    static bool asked[64] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64) {
        if (!asked[dev]) {
            using Cfg = TcCfg<128, 1, 1, 0>;
            auto kernel = tree_attention_tc_kernel<128, 1, 1, 1, 0>;
            const bool ok = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes) == cudaSuccess;
            for (int c = 2; ok && c <= kMaxClusterSplits; ++c) {
                cudaLaunchAttribute attr = {};
                attr.id = cudaLaunchAttributeClusterDimension;
                attr.val.clusterDim.x = c, attr.val.clusterDim.y = 1, attr.val.clusterDim.z = 1;
                cudaLaunchConfig_t cfg = {};
                cfg.gridDim = dim3(c, 1, 1), cfg.blockDim = dim3(Cfg::kThreads, 1, 1), cfg.dynamicSmemBytes = Cfg::kSmemBytes;
                cfg.attrs = &attr, cfg.numAttrs = 1;
                int clusters = 0;
                if (cudaOccupancyMaxActiveClusters(&clusters, kernel, &cfg) == cudaSuccess && clusters > 0) table[dev][c] = clusters * c;
            }
            cudaGetLastError();
            asked[dev] = true;
        }
        if (table[dev][s] > 0) return table[dev][s];
    } else {
        cudaGetLastError();
    }
    return 8 * (16 / s) * s;
}

// The wide path's split count (more than a cluster holds), or 0 where the path is not taken.  Shapes only: the workspace
// query depends on nothing else.
static int tc_wide_splits(int B, int T, int Hq, int Hkv, int C) {
    const int base = B * Hkv * tc_m_groups(B, T, Hq, Hkv, C);
    const int tiles = ceil_div(C, kBN);
    if (!(base * kMaxClusterSplits * 2 <= 148 && tiles >= 384 && tc_nm(B, T, Hq, Hkv, C) == 2)) return 0;
    int s = 148 / base;  // one wave
    if (s > 64) s = 64;
    return s > tiles / 2 ? tiles / 2 : s;
}

static int tc_splits(int B, int T, int Hq, int Hkv, int C) {
    if (const int wide = tc_wide_splits(B, T, Hq, Hkv, C)) return wide;
    const int base = B * Hkv * tc_m_groups(B, T, Hq, Hkv, C);
    const int tiles = ceil_div(C, kBN);
    int max_by_len = tiles / 2;
    if (max_by_len < 1) max_by_len = 1;
    int best = 1;
    double best_cost = 1e30;
    for (int s = 1; s <= kMaxClusterSplits && s <= max_by_len; ++s) {
        const int resident = tc_resident_ctas(s);
        const double waves = (double)ceil_div(base * s, resident);
        double cost = waves * (10.0 + ceil_div(tiles, s)) * (1.0 + 0.03 * (s - 1));
        // an unsplit grid of more CTAs than SMs runs as half-SM CTAs where the rows allow it (see the dispatch below): two
        // per SM at once, each streaming at half the rate
        if (s == 1 && base > 148 && (Hq / Hkv) * T <= 64) cost = ceil_div(base, 296) * (10.0 + 2.0 * tiles);
        if (cost < best_cost - 1e-12) best_cost = cost, best = s;
    }
    return best;
}

// Copies of the query rows inside the one row tile (see the kernel): 4 up to 32 rows, 2 up to 64, else 1.
static int tc_rep(int T, int Hq, int Hkv) {
    const int R = (Hq / Hkv) * T;
    return R <= 32 ? 4 : (R <= 64 ? 2 : 1);
}

// Turns (see the kernel): a single row tile per CTA, of 65..128 rows, with enough tiles per CTA is shared by two softmax groups.
static int tc_turns(int B, int T, int Hq, int Hkv, int C) {
    const int R = (Hq / Hkv) * T;
    if (R <= 64 || tc_nm(B, T, Hq, Hkv, C) == 2) return 1;
    const int tiles_per_cta = ceil_div(ceil_div(C, kBN), tc_splits(B, T, Hq, Hkv, C));
    return tiles_per_cta >= 8 ? 2 : 1;
}

size_t tc_workspace_bytes(int B, int T, int Hq, int Hkv, int d, int C) {
    const int s = tc_wide_splits(B, T, Hq, Hkv, C);  // (two row tiles per CTA: no row copies, no turns)
    return s == 0 ? 0 : round_up((size_t)B * Hq * T * s * (d + 2) * sizeof(float), 256);
}

template <int D, int NM, int REP, int TC, int PUSH, int ROWS>
static s4c_status launch_tc_layout(const void* q, const void* k, const void* v, const TcParams& prm, int B, cudaStream_t stream) {
    using Cfg = TcCfg<D, NM, TC, PUSH>;
    static bool configured[64] = {};  // the opt-ins (dynamic shared memory, cluster size) are per device
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return S4C_ERR_CUDA;
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(tree_attention_tc_kernel<D, NM, REP, TC, PUSH, ROWS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 Cfg::kSmemBytes) != cudaSuccess)
            return S4C_ERR_CUDA;
        configured[dev] = true;
    }
    CUtensorMap mq, mk, mv;
    // rows of the 2-D view of a cache: every slot of every (sequence, KV head), or of every (page, KV head)
    const uint64_t kv_rows = prm.block_table ? (uint64_t)prm.n_pages * prm.Hkv * prm.page_tiles * kBN : (uint64_t)B * prm.Hkv * prm.C;
    if (!make_map(&mq, q, (uint64_t)B * prm.Hq * prm.T, D, prm.q_box_rows) ||
        !(D == 128 ? make_map_halves(&mk, k, kv_rows, kBN) : make_map(&mk, k, kv_rows, D, kBN)) ||
        !(D == 128 ? make_map_halves(&mv, v, kv_rows, kBN) : make_map(&mv, v, kv_rows, D, kBN)))
        return S4C_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(prm.splits, prm.m_groups * prm.Hkv, B);
    cfg.blockDim = dim3(Cfg::kThreads, 1, 1);
    cfg.dynamicSmemBytes = Cfg::kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attrs[2];
    int na = 0;
    attrs[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
    if (prm.mode == kModeCluster) {
        attrs[na].id = cudaLaunchAttributeClusterDimension;
        attrs[na].val.clusterDim.x = prm.splits;
        attrs[na].val.clusterDim.y = 1;
        attrs[na].val.clusterDim.z = 1;
        ++na;
    }
    cfg.attrs = attrs;
    cfg.numAttrs = na;
    if (cudaLaunchKernelEx(&cfg, tree_attention_tc_kernel<D, NM, REP, TC, PUSH, ROWS>, mq, mk, mv, prm) != cudaSuccess) {
        cudaGetLastError();
        return S4C_ERR_CUDA;
    }
    return S4C_OK;
}

template <int D, int NM, int REP, int TC, int PUSH>
static s4c_status launch_tc(const void* q, const void* k, const void* v, const TcParams& prm, int B, cudaStream_t stream) {
    return prm.out_rows ? launch_tc_layout<D, NM, REP, TC, PUSH, 1>(q, k, v, prm, B, stream)
                        : launch_tc_layout<D, NM, REP, TC, PUSH, 0>(q, k, v, prm, B, stream);
}

// `span` (<= C) is the number of slots the launch is shaped for: the host's bound on the live length (committed tokens
// plus tree slots) where the caller gave one, else the capacity.  It steers the choices below and nothing else: the kernel
// deals out the tiles of the true length, whatever that is.
s4c_status tree_attention_tc(const void* q, const void* k, const void* v, const int32_t* cache_len,
                             const int32_t* parent, const int32_t* n_nodes, void* out, int B, int T, int Hq, int Hkv,
                             int d, int C_slots, int span, float scale, int32_t* status, void* ws, cudaStream_t stream,
                             int wait_limit_us, int withhold_tile, const TcPaging* paging, int out_rows) {
    TcParams prm;
    prm.out_rows = out_rows;
    prm.cache_len = cache_len, prm.parent = parent, prm.n_nodes = n_nodes;
    prm.out = static_cast<__nv_bfloat16*>(out), prm.ws = static_cast<float*>(ws), prm.status = status;
    prm.T = T, prm.Hq = Hq, prm.Hkv = Hkv, prm.C = C_slots;
    prm.wait_limit = wait_limit_us > 0 ? 2000ll * wait_limit_us : kWaitLimitCycles;  // about 2 cycles per nanosecond
    prm.withhold_tile = withhold_tile;
    prm.block_table = paging ? paging->block_table : nullptr;
    prm.max_blocks = paging ? paging->max_blocks : 0;
    prm.page_tiles = paging ? paging->page_size / kBN : 1;
    prm.n_pages = paging ? paging->n_pages : 0;
    const int C = span;  // every choice below is made for the live span
    const int nm = tc_nm(B, T, Hq, Hkv, C);
    prm.m_groups = tc_m_groups(B, T, Hq, Hkv, C);
    prm.splits = tc_splits(B, T, Hq, Hkv, C);
    const int rep = tc_rep(T, Hq, Hkv), turns = tc_turns(B, T, Hq, Hkv, C);
    // copies and turns merge like splits, so a single split with either still takes the (one-CTA) cluster path
    prm.mode = prm.splits > kMaxClusterSplits ? kModeWorkspace
                                              : (prm.splits == 1 && rep == 1 && turns == 1 ? kModeDirect : kModeCluster);
    const int R = (Hq / Hkv) * T;
    prm.q_box_rows = R >= kBM ? kBM : (int)round_up((size_t)R, 8);
    prm.scale_log2 = scale * 1.4426950408889634f;
    s4c_status st;
    // pushed partials (see the kernel): few rows, few tiles per CTA -- where the end of a launch, not its streaming, decides
    const int tiles_per_cta = ceil_div(ceil_div(C, kBN), prm.splits);
    const bool push = prm.mode == kModeCluster && nm == 1 && turns == 1 && tiles_per_cta <= 16 &&
                      ceil_div(R, prm.splits) * prm.splits * (d + 4) * 4 <= 32768;
    // half-SM CTAs: grids of more CTAs than SMs that need no merge (a second wave of a few CTAs costs a whole pass;
    // 256 CTAs at L=2048: 54.6 -> 49.6 us, 160 CTAs at L=512: 22.3 -> 17.8 us)
    const bool half = prm.splits == 1 && nm == 1 && turns == 1 && B * Hkv * prm.m_groups > 148;
#define S4C_TC_DISPATCH(DD)                                                                    \
    (half         ? (rep == 4   ? launch_tc<DD, 1, 4, 1, 2>(q, k, v, prm, B, stream)            \
                     : rep == 2 ? launch_tc<DD, 1, 2, 1, 2>(q, k, v, prm, B, stream)            \
                                : launch_tc<DD, 1, 1, 1, 2>(q, k, v, prm, B, stream))           \
     : nm == 2    ? launch_tc<DD, 2, 1, 1, 0>(q, k, v, prm, B, stream)                          \
     : turns == 2 ? launch_tc<DD, 1, 1, 2, 0>(q, k, v, prm, B, stream)                          \
     : rep == 4   ? (push ? launch_tc<DD, 1, 4, 1, 1>(q, k, v, prm, B, stream)                  \
                          : launch_tc<DD, 1, 4, 1, 0>(q, k, v, prm, B, stream))                 \
     : rep == 2   ? (push ? launch_tc<DD, 1, 2, 1, 1>(q, k, v, prm, B, stream)                  \
                          : launch_tc<DD, 1, 2, 1, 0>(q, k, v, prm, B, stream))                 \
                  : launch_tc<DD, 1, 1, 1, 0>(q, k, v, prm, B, stream)) /* more than 64 rows never fit the receive area */
    st = d == 128 ? S4C_TC_DISPATCH(128) : S4C_TC_DISPATCH(64);
#undef S4C_TC_DISPATCH
    if (st != S4C_OK) return st;
    if (prm.mode == kModeWorkspace)
        return tree_attention_combine(ws, cache_len, parent, n_nodes, out, B, T, Hq, d, prm.C, prm.splits * rep * turns, S4C_BF16,
                                      stream, out_rows);
    return S4C_OK;
}

}  // namespace s4c
