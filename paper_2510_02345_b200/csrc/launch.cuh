// Kernel launches of the forward chain.  Every kernel of the chain is launched with programmatic
// stream serialization and calls pdl_wait() before it touches anything an earlier kernel wrote: its
// blocks may be scheduled while the previous kernel is still draining, and wait there until that
// kernel has completed and its writes are visible.  The persistent kernels (grids of at most one block
// per SM) put the wait after their set-up (barriers, tensor-memory allocation) and then call
// pdl_release_dependents(), so that the next kernel's blocks take each SM as soon as a block of this
// grid leaves it and have their own set-up done by the time the grid has finished.  Nothing else
// overlaps; what is saved is the launch gap and the set-up between the kernels of one forward.
#pragma once

#include <atomic>

#include <cuda_runtime.h>

namespace cmoe {

// The dynamic shared-memory limit of a kernel is a per-device attribute: `done` is the calling site's record
// (one bit per device ordinal) of the devices it has been set on.  The current device is the one the launch
// that follows goes to.
template <typename Kern>
inline cudaError_t ensure_dynamic_smem(Kern kern, size_t bytes, std::atomic<unsigned long long>& done) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const unsigned long long bit = 1ull << (dev & 63);
  if (done.load(std::memory_order_relaxed) & bit) return cudaSuccess;
  e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e != cudaSuccess) return e;
  done.fetch_or(bit, std::memory_order_relaxed);
  return cudaSuccess;
}

// Blocks until the kernels this one depends on have completed (a no-op for an ordinary launch).
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Lets the next kernel of the chain be scheduled before this grid has finished (its blocks still wait in
// pdl_wait() for this grid's completion).  Called after this kernel's own pdl_wait(), so at most two kernels
// of the chain are on the device, and only by grids that are resident as a whole (no more blocks than SMs):
// every block of such a grid already has its SM, so a dependent block can only take an SM that a block of this
// grid has left, never one that a block of this grid still waits for.
__device__ __forceinline__ void pdl_release_dependents() {
  uint32_t nsm;
  asm("mov.u32 %0, %%nsmid;" : "=r"(nsm));
  if (gridDim.x * gridDim.y * gridDim.z <= nsm) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

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
