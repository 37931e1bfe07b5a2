// Programmatic dependent launch for the kernels of one training iteration.  A kernel launched
// through OverlapLaunch may be made resident while its predecessor in the stream is still
// draining; it sets up what depends on no other kernel (barriers, tensor memory, descriptor
// prefetch), then calls grid_dependency_wait(), which returns once the predecessor has finished
// and its writes are visible.  Every such kernel calls the wait in every thread before its first
// access to global memory, and releases its own successor only after that wait, so a kernel's
// set-up never overlaps anything older than its direct predecessor.
#pragma once
#include <cuda_runtime.h>

namespace retexo {

__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Launch configuration with the stream-serialisation attribute set (and, for cluster_x > 1, the cluster
// shape).  Only for kernels that call grid_dependency_wait().
struct OverlapLaunch {
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[2];
    OverlapLaunch(dim3 grid, dim3 block, size_t smem, cudaStream_t st, unsigned cluster_x = 1) {
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = cluster_x; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
        cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
        cfg.attrs = attr;
        cfg.numAttrs = cluster_x > 1 ? 2 : 1;
    }
};

}  // namespace retexo
