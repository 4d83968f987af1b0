// Kernel launches with programmatic dependent launch: a kernel launched this way may become
// resident while the previous kernel of the stream is still running, which hides its launch
// latency and prologue.  A kernel launched this way calls pdl_wait() before its first access
// to global memory (it returns once the previous kernel has completed and its writes are
// visible) and pdl_launch_dependents() at the top.  Used for the clear kernel and the scoring
// kernel behind it (202 instead of 207 us per layer on the 32K GQA workload, 93 instead of
// 97 us on the 16K MHA one) and for the gather kernel behind the one-CTA select kernel (another
// 1.5 us per layer).  The select kernel itself is launched the plain way: launched early as
// well it gains 0.6-1 us alone, but with both early the layer takes 7.5 us longer, and a gather
// kernel that lets the next call's kernels in early costs 1.5 us (both measured).
#pragma once
#include <cuda_runtime.h>

namespace snapkv {

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                       cudaStream_t stream, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace snapkv
