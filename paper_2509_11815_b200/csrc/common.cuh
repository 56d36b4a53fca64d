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

#define SPECVLM_REQUIRE(cond, msg)                                              \
  do {                                                                          \
    if (!(cond)) return ::specvlm::fail(SPECVLM_ERR_INVALID_ARG, std::string(msg)); \
  } while (0)

}  // namespace specvlm
