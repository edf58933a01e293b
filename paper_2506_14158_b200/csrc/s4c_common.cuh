// Shared host/device helpers of libs4c (not part of the public ABI).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "s4c.h"

#define S4C_MAX_T 128
#define S4C_MASK_WORDS 4  // S4C_MAX_T / 32

#define S4C_RETURN_IF_CUDA_ERROR()                         \
    do {                                                   \
        if (cudaGetLastError() != cudaSuccess) return S4C_ERR_CUDA; \
    } while (0)

namespace s4c {

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }
static inline size_t round_up(size_t x, size_t m) { return (x + m - 1) / m * m; }
static inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
static inline size_t dtype_size(s4c_dtype dt) { return dt == S4C_F32 ? 4 : 2; }

// Checks one sequence's tree and fills, for every node i < n, the bitmask of the nodes on the path
// root..i (bit t of anc[i] set iff t is i or an ancestor of i) and its depth.  Runs on one CTA; the
// caller has loaded parent[] into `par` (shared memory) and synchronised.  Returns the S4C_SEQ_*
// flags (0 = well formed); on a malformed tree the masks are not to be used.
__device__ __forceinline__ int build_ancestor_masks(const int32_t* par, int n, int T, uint32_t (*anc)[S4C_MASK_WORDS],
                                                    int* depth, int* flag_smem) {
    if (threadIdx.x == 0) *flag_smem = (n < 1 || n > T) ? S4C_SEQ_BAD_PARENT : 0;
    __syncthreads();
    if (*flag_smem) return *flag_smem;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const int p = par[i];
        if ((i == 0 && p != -1) || (i > 0 && (p < 0 || p >= i))) atomicOr(flag_smem, S4C_SEQ_BAD_PARENT);
    }
    __syncthreads();
    if (*flag_smem) return *flag_smem;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        uint32_t m[S4C_MASK_WORDS] = {0, 0, 0, 0};
        int dep = -1;
        // parent[t] < t was checked, so this chain ends after at most i + 1 steps
        for (int t = i, guard = 0; t >= 0 && guard <= i; t = par[t], ++guard) {
            m[t >> 5] |= 1u << (t & 31);
            ++dep;
        }
#pragma unroll
        for (int w = 0; w < S4C_MASK_WORDS; ++w) anc[i][w] = m[w];
        if (depth) depth[i] = dep;
    }
    __syncthreads();
    return 0;
}

}  // namespace s4c
