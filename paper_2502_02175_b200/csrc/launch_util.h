// Launch helper with programmatic dependent launch: a kernel launched through it may begin while its
// predecessor on the stream is still running, so that it can fetch data no earlier kernel writes
// (weights) ahead of time.  Such a kernel must execute pdl_wait() before it reads or writes anything
// an earlier kernel touches, and should execute pdl_trigger() once it has issued its first loads.
#pragma once
#include <cuda_runtime.h>

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
#ifdef VLAC_NO_PDL
  cfg.numAttrs = 0;
#endif
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
