// Programmatic dependent launch: a kernel launched through launch_pdl may be scheduled while its
// predecessor in the stream is still running (once the predecessor has called pdl_trigger in all its
// CTAs, or has finished), so its set-up -- barrier initialisation, TMEM allocation, shared-memory
// carving -- overlaps the predecessor's tail.  Such a kernel must call pdl_wait() before it reads
// anything the predecessor writes or overwrites anything the predecessor reads; pdl_wait returns
// when the predecessor grid has completed and its writes are visible.  Without the launch attribute
// (or after a copy) both calls are no-ops, so kernels carry them unconditionally.
#pragma once

#include <cuda_runtime.h>

namespace kvb {

// pdl = false launches without the attribute (a context's debug option; the kernels' waits are then no-ops)
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(bool pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif

}  // namespace kvb
