// Programmatic dependent launch: every kernel of the library is launched with the stream-serialisation
// attribute and begins with `pdl_sync()`.  The kernel that follows in the stream may then be set up and its
// blocks made resident while this one still runs (as soon as all blocks of this one have started); its own
// `pdl_sync()` holds it until this one has completed and its writes are visible.  What is saved is the
// launch gap between consecutive kernels of a step.
#pragma once
#include <cuda_runtime.h>

#include <utility>

namespace ngc {

__device__ __forceinline__ void pdl_sync() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

template <typename... KArgs, typename... Args>
cudaError_t launch_k(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args &&...args) {
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
  return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

}  // namespace ngc
