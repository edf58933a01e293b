// s4c_launch_floor: an empty kernel with the launch shape of a tree-attention launch -- a measurement aid.
//
// A verify step is a chain of small dependent launches (one attention launch per decoder layer); at short contexts
// each launch moves a few megabytes and its fixed costs decide the time.  This kernel does what every such launch
// must do and nothing else: it becomes resident with the same block size, dynamic shared memory and cluster shape,
// initialises a few mbarriers, allocates and frees tensor memory, waits for the previous launch of the stream
// (griddepcontrol.wait), reads one word of global memory (as the attention kernel reads the cache length before it
// can request its first tile), releases its dependents, takes the given number of cluster barriers and leaves.
// Timed in a CUDA graph of as many nodes as the step has layers it gives the floor under one attention launch.
#include <cuda_runtime.h>
#include <stdint.h>

#include "s4c_common.cuh"

namespace s4c {

__global__ void launch_floor_kernel(int tmem_cols, int cluster_syncs, const int32_t* __restrict__ word, int32_t* __restrict__ sink) {
    extern __shared__ __align__(16) unsigned char floor_smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(floor_smem);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(floor_smem + 256);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == 0) {
        if (lane < 16) {
            const uint32_t bar = (uint32_t)__cvta_generic_to_shared(bars + lane);
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(1u));
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1 && tmem_cols > 0) {
        const uint32_t slot = (uint32_t)__cvta_generic_to_shared(tmem_slot);
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"((uint32_t)tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int32_t w = word ? *word : 0;  // the first dependent read of a real launch
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (w == 0x7fffffff && sink) *sink = w;  // keeps the load alive; never true for a cache length
    for (int i = 0; i < cluster_syncs; ++i) {
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    }
    __syncthreads();
    if (warp == 1 && tmem_cols > 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(*tmem_slot), "r"((uint32_t)tmem_cols) : "memory");
    }
}

}  // namespace s4c

extern "C" s4c_status s4c_launch_floor(int ctas, int cluster, int threads, int smem_bytes, int tmem_cols, int cluster_syncs,
                                       int dependent_launch, const int32_t* word, int32_t* sink, s4c_stream_t stream_) {
    using namespace s4c;
    if (ctas < 1 || cluster < 1 || cluster > 8 || ctas % cluster != 0 || threads < 64 || threads > 1024 || threads % 32 != 0)
        return S4C_ERR_SHAPE;
    if (smem_bytes < 512 || smem_bytes > 227 * 1024 || cluster_syncs < 0 || cluster_syncs > 16) return S4C_ERR_SHAPE;
    if (tmem_cols != 0 && tmem_cols != 32 && tmem_cols != 64 && tmem_cols != 128 && tmem_cols != 256 && tmem_cols != 512)
        return S4C_ERR_SHAPE;
    if (cluster_syncs > 0 && cluster == 1) cluster_syncs = 0;
    if (cudaFuncSetAttribute(launch_floor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) != cudaSuccess) {
        cudaGetLastError();
        return S4C_ERR_CUDA;
    }
    // CTAs that share an SM must all find their tensor-memory columns: a CTA that waited for columns held by a CTA
    // which in turn waits at a cluster barrier could wait for ever
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, launch_floor_kernel, threads, smem_bytes) != cudaSuccess) {
        cudaGetLastError();
        return S4C_ERR_CUDA;
    }
    if (per_sm < 1 || (long long)per_sm * tmem_cols > 512) return S4C_ERR_UNSUPPORTED;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ctas, 1, 1), cfg.blockDim = dim3(threads, 1, 1), cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = static_cast<cudaStream_t>(stream_);
    cudaLaunchAttribute attrs[2];
    int na = 0;
    if (dependent_launch) {
        attrs[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attrs[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    if (cluster > 1) {
        attrs[na].id = cudaLaunchAttributeClusterDimension;
        attrs[na].val.clusterDim.x = cluster, attrs[na].val.clusterDim.y = 1, attrs[na].val.clusterDim.z = 1;
        ++na;
    }
    cfg.attrs = attrs, cfg.numAttrs = na;
    if (cudaLaunchKernelEx(&cfg, launch_floor_kernel, tmem_cols, cluster_syncs, word, sink) != cudaSuccess) {
        cudaGetLastError();
        return S4C_ERR_CUDA;
    }
    return S4C_OK;
}
