// s4c_tree_attention: argument validation and kernel selection.
#include <math.h>

#include "tree_attention.cuh"

namespace s4c {

static s4c_status check_shapes(int B, int T, int Hq, int Hkv, int d, int C, s4c_dtype dt) {
    if (dt != S4C_F32 && dt != S4C_BF16) return S4C_ERR_DTYPE;
    if (B < 0 || B > 65535 || T < 1 || T > S4C_MAX_T || Hq < 1 || Hkv < 1 || Hq > 65535 || Hq % Hkv != 0 || C < 1)
        return S4C_ERR_SHAPE;
    if (d != 64 && d != 128) return S4C_ERR_SHAPE;
    return S4C_OK;
}

}  // namespace s4c

extern "C" size_t s4c_tree_attention_workspace_bytes(int B, int T, int Hq, int Hkv, int d, int C, s4c_dtype dt) {
    using namespace s4c;
    if (check_shapes(B, T, Hq, Hkv, d, C, dt) != S4C_OK || B == 0) return 0;
    if (tc_supported(T, Hq, Hkv, d, dt)) return tc_workspace_bytes(B, T, Hq, Hkv, d, C);
    return simt_workspace_bytes(B, T, Hq, d, C);
}

namespace s4c {
static s4c_status attention_run(const void* q, const void* k_cache, const void* v_cache, const int32_t* cache_len,
                                const int32_t* parent, const int32_t* n_nodes, void* out, int B, int T, int Hq, int Hkv, int d, int C,
                                int max_cache_len, s4c_dtype dt, float scale, int32_t* status, void* workspace,
                                size_t workspace_bytes, s4c_stream_t stream_, int out_rows) {
    const s4c_status st = check_shapes(B, T, Hq, Hkv, d, C, dt);
    if (st != S4C_OK) return st;
    if (!q || !k_cache || !v_cache || !cache_len || !parent || !out) return S4C_ERR_NULL;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(out)) return S4C_ERR_ALIGN;
    if (!(scale >= 0.f) || isinf(scale) || max_cache_len < 0) return S4C_ERR_SHAPE;
    if (out_rows && !tc_supported(T, Hq, Hkv, d, dt)) return S4C_ERR_UNSUPPORTED;  // the row layout exists on the tensor-core path (bf16) only
    if (B == 0) return S4C_OK;
    if (scale == 0.f) scale = 1.f / sqrtf((float)d);
    const size_t need = s4c_tree_attention_workspace_bytes(B, T, Hq, Hkv, d, C, dt);
    if (need > 0 && (!workspace || workspace_bytes < need || !aligned256(workspace))) return S4C_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    // the slots the launch is shaped for: the host's bound on the committed lengths plus the tree, where one was given
    const int span = (max_cache_len > 0 && (long long)max_cache_len + T < (long long)C) ? max_cache_len + T : C;
    if (tc_supported(T, Hq, Hkv, d, dt))
        return tree_attention_tc(q, k_cache, v_cache, cache_len, parent, n_nodes, out, B, T, Hq, Hkv, d, C, span, scale,
                                 status, workspace, stream, 0, -1, nullptr, out_rows);
    return tree_attention_simt(q, k_cache, v_cache, cache_len, parent, n_nodes, out, B, T, Hq, Hkv, d, C, span, dt, scale,
                               status, workspace, stream);
}
}  // namespace s4c

extern "C" s4c_status s4c_tree_attention(const void* q, const void* k_cache, const void* v_cache,
                                         const int32_t* cache_len, const int32_t* parent, const int32_t* n_nodes,
                                         void* out, int B, int T, int Hq, int Hkv, int d, int C, int max_cache_len,
                                         s4c_dtype dt, float scale, int32_t* status, void* workspace,
                                         size_t workspace_bytes, s4c_stream_t stream) {
    return s4c::attention_run(q, k_cache, v_cache, cache_len, parent, n_nodes, out, B, T, Hq, Hkv, d, C, max_cache_len, dt, scale, status,
                              workspace, workspace_bytes, stream, 0);
}

extern "C" s4c_status s4c_tree_attention_rows(const void* q, const void* k_cache, const void* v_cache,
                                              const int32_t* cache_len, const int32_t* parent, const int32_t* n_nodes,
                                              void* out_rows, int B, int T, int Hq, int Hkv, int d, int C, int max_cache_len,
                                              s4c_dtype dt, float scale, int32_t* status, void* workspace,
                                              size_t workspace_bytes, s4c_stream_t stream) {
    return s4c::attention_run(q, k_cache, v_cache, cache_len, parent, n_nodes, out_rows, B, T, Hq, Hkv, d, C, max_cache_len, dt, scale,
                              status, workspace, workspace_bytes, stream, 1);
}

// Paged caches: pages [n_pages, Hkv, page_size, d] addressed through a block table [B, max_blocks].
extern "C" s4c_status s4c_tree_attention_paged(const void* q, const void* k_pages, const void* v_pages,
                                               const int32_t* block_table, const int32_t* cache_len,
                                               const int32_t* parent, const int32_t* n_nodes, void* out, int B, int T,
                                               int Hq, int Hkv, int d, int n_pages, int page_size, int max_blocks,
                                               int max_cache_len, s4c_dtype dt, float scale, int32_t* status,
                                               void* workspace, size_t workspace_bytes, s4c_stream_t stream_) {
    using namespace s4c;
    if (n_pages < 1 || max_blocks < 1 || page_size < 64 || page_size % 64 != 0) return S4C_ERR_SHAPE;
    if ((long long)max_blocks * page_size > 0x7fffffffll || (long long)n_pages * Hkv * page_size > 0x7fffffffll) return S4C_ERR_SHAPE;
    const int C = max_blocks * page_size;  // what a sequence can hold
    const s4c_status st = check_shapes(B, T, Hq, Hkv, d, C, dt);
    if (st != S4C_OK) return st;
    if (!q || !k_pages || !v_pages || !block_table || !cache_len || !parent || !out) return S4C_ERR_NULL;
    if (!aligned16(q) || !aligned16(k_pages) || !aligned16(v_pages) || !aligned16(out)) return S4C_ERR_ALIGN;
    if (!(scale >= 0.f) || isinf(scale) || max_cache_len < 0) return S4C_ERR_SHAPE;
    if (dt != S4C_BF16) return S4C_ERR_UNSUPPORTED;  // paged caches are served by the tensor-core kernel only
    if (B == 0) return S4C_OK;
    if (scale == 0.f) scale = 1.f / sqrtf((float)d);
    const size_t need = s4c_tree_attention_workspace_bytes(B, T, Hq, Hkv, d, C, dt);
    if (need > 0 && (!workspace || workspace_bytes < need || !aligned256(workspace))) return S4C_ERR_WORKSPACE;
    const int span = (max_cache_len > 0 && (long long)max_cache_len + T < (long long)C) ? max_cache_len + T : C;
    const TcPaging paging = {block_table, max_blocks, page_size, n_pages};
    return tree_attention_tc(q, k_pages, v_pages, cache_len, parent, n_nodes, out, B, T, Hq, Hkv, d, C, span, scale, status,
                             workspace, static_cast<cudaStream_t>(stream_), 0, -1, &paging);
}

// The bounded waits of the tensor-core kernel, exercised: the same launch as s4c_tree_attention, except that the copy
// producer of every CTA never requests cache tile `withhold_tile` of its range and a wait gives up after `limit_us`
// microseconds.  The consumers of that tile run out of time with nothing in flight, every role leaves its loop, and the
// kernel returns normally with S4C_SEQ_TIMEOUT in status[b] and `out` untouched.
extern "C" s4c_status s4c_selftest_attention_timeout(const void* q, const void* k_cache, const void* v_cache,
                                                     const int32_t* cache_len, const int32_t* parent, void* out, int B,
                                                     int T, int Hq, int Hkv, int d, int C, int max_cache_len,
                                                     int withhold_tile, int limit_us, int32_t* status,
                                                     s4c_stream_t stream_) {
    using namespace s4c;
    const s4c_status st = check_shapes(B, T, Hq, Hkv, d, C, S4C_BF16);
    if (st != S4C_OK) return st;
    if (!q || !k_cache || !v_cache || !cache_len || !parent || !out || !status) return S4C_ERR_NULL;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(out)) return S4C_ERR_ALIGN;
    if (B == 0 || max_cache_len < 0 || withhold_tile < 0 || limit_us < 1 || limit_us > 100000) return S4C_ERR_SHAPE;
    if (s4c_tree_attention_workspace_bytes(B, T, Hq, Hkv, d, C, S4C_BF16) != 0) return S4C_ERR_UNSUPPORTED;  // in-cluster merge only
    const int span = (max_cache_len > 0 && (long long)max_cache_len + T < (long long)C) ? max_cache_len + T : C;
    return tree_attention_tc(q, k_cache, v_cache, cache_len, parent, nullptr, out, B, T, Hq, Hkv, d, C, span,
                             1.f / sqrtf((float)d), status, nullptr, static_cast<cudaStream_t>(stream_), limit_us, withhold_tile);
}
