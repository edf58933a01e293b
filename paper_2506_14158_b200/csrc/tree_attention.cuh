// Internal interface between the s4c_tree_attention dispatcher and its kernel families.
#pragma once
#include "s4c_common.cuh"

namespace s4c {

// CUDA-core path (float32 inputs; fallback for bf16 shapes the tensor-core path does not take).
size_t simt_workspace_bytes(int B, int T, int Hq, int d, int C);
s4c_status tree_attention_simt(const void* q, const void* k, const void* v, const int32_t* cache_len,
                               const int32_t* parent, const int32_t* n_nodes, void* out, int B, int T, int Hq, int Hkv,
                               int d, int C, int span, s4c_dtype dt, float scale, int32_t* status, void* ws,
                               cudaStream_t stream);

// Merges split partials [B*Hq*T rows][splits][d + 2] (unnormalised output, running max in base-2 units, sum).
s4c_status tree_attention_combine(const void* ws, const int32_t* cache_len, const int32_t* parent, const int32_t* n_nodes,
                                  void* out, int B, int T, int Hq, int d, int C, int splits, s4c_dtype dt,
                                  cudaStream_t stream, int out_rows = 0 /* 1: out is [B,T,Hq,d] */);

// Paged caches: pages [n_pages, Hkv, page_size, d] and a block table [B, max_blocks] (page_size a multiple of 64 slots).
struct TcPaging {
    const int32_t* block_table;
    int max_blocks, page_size, n_pages;
};

// Tensor-core path (bf16, d in {64, 128}): tcgen05 / TMEM / TMA.
bool tc_supported(int T, int Hq, int Hkv, int d, s4c_dtype dt);
size_t tc_workspace_bytes(int B, int T, int Hq, int Hkv, int d, int C);
s4c_status tree_attention_tc(const void* q, const void* k, const void* v, const int32_t* cache_len,
                             const int32_t* parent, const int32_t* n_nodes, void* out, int B, int T, int Hq, int Hkv,
                             int d, int C, int span, float scale, int32_t* status, void* ws, cudaStream_t stream,
                             int wait_limit_us = 0 /* 0: the default of about 200 ms */, int withhold_tile = -1 /* self-test only */,
                             const TcPaging* paging = nullptr /* nullptr: contiguous caches of C slots */,
                             int out_rows = 0 /* 1: out is [B,T,Hq,d] instead of [B,Hq,T,d] */);

}  // namespace s4c
