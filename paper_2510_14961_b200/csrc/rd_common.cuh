// Pieces every kernel file of the library uses: programmatic dependent launch.
//
// The kernels of one step form a chain on one stream.  Each is launched with the programmatic
// stream-serialization attribute: it may start while its predecessor still runs, must call
// pdl_wait() before it reads anything an earlier kernel wrote or writes anything an earlier kernel
// may still read, and calls pdl_trigger() at its start so that its own successor can be scheduled
// early.  pdl_wait() returns once the predecessor has completed and its writes are visible; as
// every kernel of the chain waits before it finishes, completion is transitive along the chain.
#pragma once
#include <cuda_runtime.h>

namespace rd {

__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Start of a kernel that has nothing useful to do before its inputs are ready.
__device__ __forceinline__ void pdl_enter() { pdl_trigger(); pdl_wait(); }

// Launch `kern` on `st` as a link of the chain (`chained` false: an ordinary launch).  cluster_x > 1:
// thread-block clusters of that many CTAs along x.
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_chained_cluster(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                                 cudaStream_t st, bool chained, unsigned cluster_x, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    unsigned n = 0;
    if (chained) {
        at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[n].val.programmaticStreamSerializationAllowed = 1;
        n++;
    }
    if (cluster_x > 1) {
        at[n].id = cudaLaunchAttributeClusterDimension;
        at[n].val.clusterDim.x = cluster_x;
        at[n].val.clusterDim.y = 1;
        at[n].val.clusterDim.z = 1;
        n++;
    }
    cfg.attrs = at;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_chained(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                         bool chained, Args... args) {
    return launch_chained_cluster(kern, grid, block, smem, st, chained, 1u, args...);
}

}  // namespace rd
