// Programmatic dependent launch, shared by the kernel files.
//
// A kernel launched with the stream-serialisation attribute may start while its predecessor in the
// stream is still draining.  Everything it does before pdl_wait (barrier set-up, tensor-memory
// allocation, descriptor prefetch, index arithmetic) must touch no global data; pdl_wait returns once
// the predecessor has completed and its writes are visible.  pdl_launch_dependents lets the successor
// do the same with respect to this kernel.
#pragma once
#include <cuda_runtime.h>

#include <cstring>
#include <utility>

namespace gl {

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Launch with the attribute set (every kernel launched this way calls pdl_wait before its first global
// access), optionally as clusters of `cluster` blocks.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, int cluster,
                       Args&&... args) {
  cudaLaunchConfig_t cfg;
  std::memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  std::memset(at, 0, sizeof(at));
  int n = 0;
  at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[n].val.programmaticStreamSerializationAllowed = 1;
  ++n;
  if (cluster > 1) {
    at[n].id = cudaLaunchAttributeClusterDimension;
    at[n].val.clusterDim.x = static_cast<unsigned>(cluster);
    at[n].val.clusterDim.y = 1;
    at[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = at;
  cfg.numAttrs = static_cast<unsigned>(n);
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

}  // namespace gl
