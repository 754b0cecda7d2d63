// Programmatic dependent launch, shared by the kernel files.
//
// A kernel launched with the stream-serialisation attribute may start while its predecessor in the
// stream is still draining.  Everything it does before pdl_wait (barrier set-up, tensor-memory
// allocation, descriptor prefetch, index arithmetic) must touch no global data; pdl_wait returns once
// the predecessor has completed and its writes are visible.  pdl_launch_dependents lets the successor
// do the same with respect to this kernel.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>
#include <cstring>
#include <utility>

namespace gl {

// Division of n < 2^31 by a divisor fixed on the host: p = ceil(log2 d), mul = ceil(2^(31+p) / d),
// n / d = umulhi(n, mul) >> (p - 1); mul = 0 stands for d = 1.  An integer division on the device costs
// some twenty-five instructions (over a hundred for 64-bit operands), and in the single-thread and
// single-warp loops of the tensor-core kernels it is a dependent chain of about 150 cycles.
struct FastDiv {
  uint32_t d, mul, shift;
  __host__ void set(int64_t divisor) {
    d = static_cast<uint32_t>(divisor);
    uint32_t pw2 = 0;
    while ((1ull << pw2) < static_cast<uint64_t>(divisor)) ++pw2;
    mul = pw2 ? static_cast<uint32_t>(((1ull << (31 + pw2)) + divisor - 1) / divisor) : 0u;
    shift = pw2 ? pw2 - 1 : 0u;
  }
  __device__ __forceinline__ uint32_t div(uint32_t n) const { return mul ? (__umulhi(n, mul) >> shift) : n; }
  __device__ __forceinline__ void divmod(uint32_t n, uint32_t& q, uint32_t& r) const { q = div(n); r = n - q * d; }
};
inline FastDiv make_fastdiv(int64_t d) {
  FastDiv fd;
  fd.set(d);
  return fd;
}
__device__ __forceinline__ uint32_t fdiv(uint32_t n, const FastDiv& fd) { return fd.div(n); }

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
