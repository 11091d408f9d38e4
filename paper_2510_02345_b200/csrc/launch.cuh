// Kernel launches of the forward chain.  Every kernel of the chain starts with pdl_wait() and is
// launched with programmatic stream serialization: the next kernel's blocks may be scheduled while
// the previous kernel is still draining, and wait at their first instruction until it has completed
// and its writes are visible.  Nothing else overlaps; what is saved is the launch gap between the
// dozen short kernels of one forward.
#pragma once

#include <cuda_runtime.h>

namespace cmoe {

// Blocks until the kernels this one depends on have completed (a no-op for an ordinary launch).
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// cluster = 2 launches thread-block clusters of two CTAs (grid.x must be even)
template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                  int cluster, Args... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  int n = 1;
  if (cluster > 1) {
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)cluster;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    n = 2;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

}  // namespace cmoe
