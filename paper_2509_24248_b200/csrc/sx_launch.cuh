// Launch helper with programmatic dependent launch: a kernel launched through sx_launch may be
// scheduled while its predecessor in the stream is still draining, so that its prologue (and,
// for the GEMMs, the first ring of weight tiles, which depend on nothing) overlaps the
// predecessor's tail.  Every kernel launched this way executes sx_pdl_wait() before it reads or
// writes anything another kernel of the stream produces or consumes; completion is therefore
// transitive along the stream exactly as with plain stream order.
#pragma once
#include <cuda_runtime.h>

#include <string.h>

#include <utility>

__device__ __forceinline__ void sx_pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void sx_pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// overlap = false launches in plain stream order (the kernel starts when its predecessor has completed; its
// griddepcontrol instructions are then no-ops).
template <typename... KArgs, typename... Args>
inline cudaError_t sx_launch_opt(bool overlap, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                 cudaStream_t st, Args &&...args) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = overlap ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
}

template <typename... KArgs, typename... Args>
inline cudaError_t sx_launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                             Args &&...args) {
  return sx_launch_opt(true, kernel, grid, block, smem, st, std::forward<Args>(args)...);
}

// The same with a thread-block cluster of `cluster` CTAs along x (grid.x must be a multiple of it).
template <typename... KArgs, typename... Args>
inline cudaError_t sx_launch_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, unsigned cluster,
                                     cudaStream_t st, Args &&...args) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = cluster;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
}
