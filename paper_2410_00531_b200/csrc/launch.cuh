// Kernel launch helper: optional programmatic dependent launch, launch counting.
#pragma once
#include <cuda_runtime.h>

#include "kernels.h"

namespace tpi {

template <typename... KArgs, typename... Args>
static inline cudaError_t launch_kernel(const LaunchCtx& c, void (*kern)(KArgs...), dim3 grid, dim3 block,
                                        size_t smem, Args... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = c.stream;
  cudaLaunchAttribute attr[1];
  if (c.pdl) {
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
  }
  if (c.launches) ++*c.launches;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

}  // namespace tpi
