// Shared host/device helpers of the tree-verification library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <string>

#include "specvlm.h"

namespace specvlm {

// Records the calling thread's last error text and returns `code`.
int fail(int code, const std::string& msg);
// Maps a CUDA runtime error to SPECVLM_ERR_CUDA (or SPECVLM_OK).
int check_cuda(cudaError_t e, const char* what);
// Number of SMs of the current device (cached per device).
int sm_count();
// Split count the attention launch uses when the descriptor leaves it to the library.
int resolve_num_splits(const specvlm_attn_desc& d);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

#ifdef __CUDACC__
// Programmatic dependent launch for the small kernels of a step. A kernel launched with
// launch_overlapped() may be scheduled while the preceding kernel on the stream is still running;
// it must call grid_dependency_sync() before it touches global memory. That call waits until the
// preceding kernel has completed and its writes are visible, and only then lets the next kernel
// be scheduled: the order of all memory effects is that of ordinary stream order, a kernel never
// runs beside anything but its immediate predecessor, and what overlaps is launch latency and
// block scheduling.
__device__ __forceinline__ void grid_dependency_sync() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <class... KArgs, class... Args>
cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

#define SPECVLM_REQUIRE(cond, msg)                                              \
  do {                                                                          \
    if (!(cond)) return ::specvlm::fail(SPECVLM_ERR_INVALID_ARG, std::string(msg)); \
  } while (0)

}  // namespace specvlm
