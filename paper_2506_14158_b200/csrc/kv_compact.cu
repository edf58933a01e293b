// s4c_kv_compact: in-place compaction of the accepted path's K/V rows (all layers) and gather of the
// accepted nodes' hidden features (Section 3.2, last paragraph; feature reuse, Section 1).
//
// Data movement only, in 16-byte words.  One thread owns one 16-byte column of one (layer, K|V, b, head)
// row set and moves it for j = 1..a in ascending order.  Because a path is strictly increasing
// (path[j] >= j), a destination slot j is never a source of a later copy, so the ascending order is
// race-free in place without a snapshot; loads are issued in batches ahead of their stores for
// memory-level parallelism.  cache_len is read by the copy kernel and rewritten by a second, tiny
// kernel ordered after it on the stream (which also gathers the features), so no CTA can observe the
// new length.
#include "s4c_common.cuh"

namespace s4c {

struct PathInfo {
    int flags;  // S4C_SEQ_*; -1 = sequence skipped (accept_len < 0)
    int a;
    int L;
};

// Same checks in both kernels, evaluated redundantly by every thread that needs them (<= 128 ints).
__device__ __forceinline__ PathInfo check_path(const int32_t* cache_len, const int32_t* path,
                                               const int32_t* accept_len, int b, int max_depth, int T, int C) {
    PathInfo r;
    r.a = accept_len[b];
    r.L = cache_len[b];
    r.flags = 0;
    if (r.a < 0) {
        r.flags = -1;
        return r;
    }
    if (r.a > max_depth) r.flags |= S4C_SEQ_DEPTH;
    if (r.L < 0 || (long long)r.L + T > (long long)C) r.flags |= S4C_SEQ_CAPACITY;
    if (r.flags) return r;
    const int32_t* p = path + (size_t)b * (max_depth + 1);
    if (p[0] != 0) r.flags |= S4C_SEQ_BAD_PATH;
    int prev = -1;
    for (int j = 0; j <= r.a; ++j) {
        const int v = p[j];
        if (v < j || v >= T || v <= prev) r.flags |= S4C_SEQ_BAD_PATH;
        prev = v;
    }
    return r;
}

constexpr int kCompactThreads = 256;
constexpr int kBatch = 4;
constexpr int kMaxTreeBlocks = S4C_MAX_T / 64 + 2;  // pages the tree slots L..L+T-1 can touch (a page holds >= 64 slots)

// Paged caches [n_pages, Hkv, page_size, d] with a block table [B, max_blocks]; table == nullptr: contiguous caches.
struct Paging {
    const int32_t* table;
    int max_blocks, page_size, n_pages;
};
// The pages of the blocks that hold the tree slots of sequence b, into `pages` (first block: L / page_size).  Returns
// S4C_SEQ_BAD_PAGE if one of them lies outside the pool or the table is too short, else 0.
__device__ __forceinline__ int load_tree_pages(const Paging& pg, int b, int L, int T, int* pages) {
    const int blk0 = L / pg.page_size, blk1 = (L + T - 1) / pg.page_size;
    int flags = 0;
    for (int i = blk0; i <= blk1; ++i) {
        int page = -1;
        if (i < pg.max_blocks) page = pg.table[(size_t)b * pg.max_blocks + i];
        if ((unsigned)page >= (unsigned)pg.n_pages) flags = S4C_SEQ_BAD_PAGE, page = 0;
        pages[i - blk0] = page;
    }
    return flags;
}

// grid: (item blocks, n_layers, B).  Items of one (layer, b): Hkv heads x {K,V} x words per row.
__global__ void __launch_bounds__(kCompactThreads)
kv_compact_rows_kernel(void* const* __restrict__ k_caches, void* const* __restrict__ v_caches,
                       const int32_t* __restrict__ cache_len, const int32_t* __restrict__ path,
                       const int32_t* __restrict__ accept_len, int max_depth, int T, int Hkv, int C,
                       int words_per_row, const Paging pg) {
    const int b = blockIdx.z, layer = blockIdx.y;
    __shared__ PathInfo info;
    __shared__ int32_t spath[S4C_MAX_T];
    __shared__ int pages[kMaxTreeBlocks];
    if (threadIdx.x == 0) {
        info = check_path(cache_len, path, accept_len, b, max_depth, T, C);
        if (pg.table && info.flags == 0) info.flags |= load_tree_pages(pg, b, info.L, T, pages);
    }
    __syncthreads();
    if (info.flags != 0 || info.a == 0) return;  // nothing to move (path[0] == 0 stays in place)
    const int a = info.a;
    for (int j = threadIdx.x; j <= a; j += blockDim.x) spath[j] = path[(size_t)b * (max_depth + 1) + j];
    __syncthreads();

    const int items = Hkv * 2 * words_per_row;
    const int item = blockIdx.x * blockDim.x + threadIdx.x;
    if (item >= items) return;
    const int w = item % words_per_row;
    const int kv = (item / words_per_row) & 1;
    const int h = item / (2 * words_per_row);
    uint4* cache = reinterpret_cast<uint4*>(kv ? v_caches[layer] : k_caches[layer]);
    // the 16-byte word of tree slot i (slot L + i of the sequence) that this thread owns
    const int blk0 = pg.table ? info.L / pg.page_size : 0;
    auto word_of = [&](int i) -> uint4* {
        if (!pg.table) return cache + (((size_t)b * Hkv + h) * C + info.L + i) * words_per_row + w;
        const int slot = info.L + i, page = pages[slot / pg.page_size - blk0];
        return cache + (((size_t)page * Hkv + h) * pg.page_size + slot % pg.page_size) * words_per_row + w;
    };

    for (int j0 = 1; j0 <= a; j0 += kBatch) {
        uint4 buf[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u)
            if (j0 + u <= a) buf[u] = *word_of(spath[j0 + u]);
#pragma unroll
        for (int u = 0; u < kBatch; ++u)
            if (j0 + u <= a) *word_of(j0 + u) = buf[u];
    }
}

// grid: (B).  Gathers the features, writes the per-sequence status and the new cache length.
__global__ void __launch_bounds__(kCompactThreads)
kv_compact_finish_kernel(int32_t* __restrict__ cache_len, const int32_t* __restrict__ path,
                         const int32_t* __restrict__ accept_len, int max_depth, int T, int C,
                         const uint4* __restrict__ feat_in, uint4* __restrict__ feat_out, int feat_words,
                         int32_t* __restrict__ status, const Paging pg) {
    const int b = blockIdx.x;
    __shared__ PathInfo info;
    if (threadIdx.x == 0) {
        info = check_path(cache_len, path, accept_len, b, max_depth, T, C);
        int pages[kMaxTreeBlocks];
        if (pg.table && info.flags == 0) info.flags |= load_tree_pages(pg, b, info.L, T, pages);
    }
    __syncthreads();
    const PathInfo r = info;
    if (threadIdx.x == 0 && status) status[b] = r.flags < 0 ? 0 : r.flags;
    if (r.flags != 0) return;
    if (feat_in && feat_out) {
        const int32_t* p = path + (size_t)b * (max_depth + 1);
        const int total = (r.a + 1) * feat_words;
        for (int i = threadIdx.x; i < total; i += blockDim.x) {
            const int j = i / feat_words, w = i - j * feat_words;
            feat_out[((size_t)b * (max_depth + 1) + j) * feat_words + w] =
                feat_in[((size_t)b * T + p[j]) * feat_words + w];
        }
    }
    __syncthreads();  // every thread has read cache_len (through `info`) before it changes
    if (threadIdx.x == 0) cache_len[b] = r.L + r.a + 1;
}

}  // namespace s4c

namespace s4c {

static s4c_status kv_compact_launch(void* const* k_caches, void* const* v_caches, int n_layers, int32_t* cache_len,
                                    const int32_t* path, const int32_t* accept_len, int max_depth, const void* feat_in,
                                    void* feat_out, int B, int T, int Hkv, int d, int C, int hid, s4c_dtype dt,
                                    int32_t* status, const Paging& pg, cudaStream_t stream) {
    if (dt != S4C_F32 && dt != S4C_BF16) return S4C_ERR_DTYPE;
    if (!cache_len || !path || !accept_len) return S4C_ERR_NULL;
    if (n_layers < 0 || B < 0 || T < 1 || T > S4C_MAX_T || Hkv < 1 || d < 1 || C < 1 || max_depth < 0 ||
        max_depth >= S4C_MAX_T || hid < 0)
        return S4C_ERR_SHAPE;
    if (n_layers > 0 && (!k_caches || !v_caches)) return S4C_ERR_NULL;
    if ((feat_in == nullptr) != (feat_out == nullptr)) return S4C_ERR_NULL;
    const size_t es = dtype_size(dt);
    if ((d * es) % 16 != 0) return S4C_ERR_SHAPE;
    if (feat_in && (hid < 1 || (hid * es) % 16 != 0)) return S4C_ERR_SHAPE;
    if (!aligned16(feat_in) || !aligned16(feat_out)) return S4C_ERR_ALIGN;
    if (B == 0) return S4C_OK;
    const int words_per_row = (int)(d * es / 16);
    if (n_layers > 0) {
        const int items = Hkv * 2 * words_per_row;
        dim3 grid(ceil_div(items, kCompactThreads), n_layers, B);
        kv_compact_rows_kernel<<<grid, kCompactThreads, 0, stream>>>(k_caches, v_caches, cache_len, path, accept_len,
                                                                      max_depth, T, Hkv, C, words_per_row, pg);
        S4C_RETURN_IF_CUDA_ERROR();
    }
    kv_compact_finish_kernel<<<B, kCompactThreads, 0, stream>>>(
        cache_len, path, accept_len, max_depth, T, C, static_cast<const uint4*>(feat_in),
        static_cast<uint4*>(feat_out), feat_in ? (int)(hid * es / 16) : 0, status, pg);
    S4C_RETURN_IF_CUDA_ERROR();
    return S4C_OK;
}

}  // namespace s4c

extern "C" s4c_status s4c_kv_compact(void* const* k_caches, void* const* v_caches, int n_layers,
                                     int32_t* cache_len, const int32_t* path, const int32_t* accept_len,
                                     int max_depth, const void* feat_in, void* feat_out, int B, int T, int Hkv,
                                     int d, int C, int hid, s4c_dtype dt, int32_t* status, s4c_stream_t stream_) {
    const s4c::Paging none = {nullptr, 0, 0, 0};
    return s4c::kv_compact_launch(k_caches, v_caches, n_layers, cache_len, path, accept_len, max_depth, feat_in, feat_out, B, T,
                                  Hkv, d, C, hid, dt, status, none, static_cast<cudaStream_t>(stream_));
}

extern "C" s4c_status s4c_kv_compact_paged(void* const* k_pages, void* const* v_pages, int n_layers,
                                           const int32_t* block_table, int32_t* cache_len, const int32_t* path,
                                           const int32_t* accept_len, int max_depth, const void* feat_in, void* feat_out,
                                           int B, int T, int Hkv, int d, int n_pages, int page_size, int max_blocks,
                                           int hid, s4c_dtype dt, int32_t* status, s4c_stream_t stream_) {
    if (!block_table) return S4C_ERR_NULL;
    if (n_pages < 1 || max_blocks < 1 || page_size < 64 || page_size % 64 != 0 ||
        (long long)max_blocks * page_size > 0x7fffffffll)
        return S4C_ERR_SHAPE;
    const s4c::Paging pg = {block_table, max_blocks, page_size, n_pages};
    return s4c::kv_compact_launch(k_pages, v_pages, n_layers, cache_len, path, accept_len, max_depth, feat_in, feat_out, B, T, Hkv,
                                  d, max_blocks * page_size, hid, dt, status, pg, static_cast<cudaStream_t>(stream_));
}
