// Internal interface between the s4c_tree_attention dispatcher and its kernel families.
#pragma once
#include "s4c_common.cuh"

namespace s4c {

// CUDA-core path (float32 inputs; fallback for bf16 shapes the tensor-core path does not take).
size_t simt_workspace_bytes(int B, int T, int Hq, int d, int C);
s4c_status tree_attention_simt(const void* q, const void* k, const void* v, const int32_t* cache_len,
                               const int32_t* parent, const int32_t* n_nodes, void* out, int B, int T, int Hq, int Hkv,
                               int d, int C, s4c_dtype dt, float scale, int32_t* status, void* ws, cudaStream_t stream);

}  // namespace s4c
