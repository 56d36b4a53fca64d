// Vocabulary-wide argmax of the target logits at every tree node (the greedy target
// token used by temperature-0 verification; part of the sampling cost of Eq. 1).
//
// One thread block per logits row. Every thread keeps the (value, lowest index) of the
// maximum among the float4 groups it streams (128-bit coalesced loads), then the pairs
// are reduced with "greater value, else lower index", which reproduces a sequential scan
// with strict '>' bit for bit. HBM-bound: V * 4 bytes per row, read once.
#include "common.cuh"

#include <limits.h>

namespace specvlm {

constexpr int kArgmaxThreads = 512;

struct Best {
  float v;
  int i;
};

__device__ __forceinline__ Best better(Best a, Best b) {
  // -0.0f == +0.0f under IEEE comparison, so signed zeros tie and the lower index wins.
  return (b.v > a.v || (b.v == a.v && b.i < a.i)) ? b : a;
}

__device__ __forceinline__ void take(Best& best, float v, int i) {
  if (v > best.v) {  // indices arrive in increasing order within a thread
    best.v = v;
    best.i = i;
  }
}

__global__ void __launch_bounds__(kArgmaxThreads)
argmax_rows_kernel(const float* __restrict__ logits, int V, int64_t row_stride,
                   int32_t* __restrict__ out) {
  const int row = blockIdx.x;
  const float* x = logits + static_cast<int64_t>(row) * row_stride;
  const float4* x4 = reinterpret_cast<const float4*>(x);
  const int n4 = V >> 2;

  Best best{-INFINITY, INT_MAX};
  // -inf never passes '>' against the initial -inf; INT_MAX then loses every index tie,
  // and an all -inf row ends as index 0 below.
  int g = threadIdx.x;
  // Four independent 16-byte loads in flight per thread per trip.
  for (; g + 3 * kArgmaxThreads < n4; g += 4 * kArgmaxThreads) {
    float4 a = __ldcs(x4 + g);
    float4 b = __ldcs(x4 + g + kArgmaxThreads);
    float4 c = __ldcs(x4 + g + 2 * kArgmaxThreads);
    float4 d = __ldcs(x4 + g + 3 * kArgmaxThreads);
    int i = g * 4;
    take(best, a.x, i); take(best, a.y, i + 1); take(best, a.z, i + 2); take(best, a.w, i + 3);
    i = (g + kArgmaxThreads) * 4;
    take(best, b.x, i); take(best, b.y, i + 1); take(best, b.z, i + 2); take(best, b.w, i + 3);
    i = (g + 2 * kArgmaxThreads) * 4;
    take(best, c.x, i); take(best, c.y, i + 1); take(best, c.z, i + 2); take(best, c.w, i + 3);
    i = (g + 3 * kArgmaxThreads) * 4;
    take(best, d.x, i); take(best, d.y, i + 1); take(best, d.z, i + 2); take(best, d.w, i + 3);
  }
  for (; g < n4; g += kArgmaxThreads) {
    float4 a = __ldcs(x4 + g);
    int i = g * 4;
    take(best, a.x, i); take(best, a.y, i + 1); take(best, a.z, i + 2); take(best, a.w, i + 3);
  }
  for (int i = (n4 << 2) + threadIdx.x; i < V; i += kArgmaxThreads) take(best, x[i], i);

#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    Best o{__shfl_xor_sync(0xffffffffu, best.v, off), __shfl_xor_sync(0xffffffffu, best.i, off)};
    best = better(best, o);
  }
  __shared__ float sv[kArgmaxThreads / 32];
  __shared__ int si[kArgmaxThreads / 32];
  if ((threadIdx.x & 31) == 0) {
    sv[threadIdx.x >> 5] = best.v;
    si[threadIdx.x >> 5] = best.i;
  }
  __syncthreads();
  if (threadIdx.x < 32) {
    Best b{-INFINITY, INT_MAX};
    if (threadIdx.x < kArgmaxThreads / 32) b = Best{sv[threadIdx.x], si[threadIdx.x]};
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      Best o{__shfl_xor_sync(0xffffffffu, b.v, off), __shfl_xor_sync(0xffffffffu, b.i, off)};
      b = better(b, o);
    }
    if (threadIdx.x == 0) out[row] = (b.i == INT_MAX) ? 0 : b.i;
  }
}

int launch_argmax(const float* logits, int rows, int V, int64_t row_stride, int32_t* out,
                  cudaStream_t stream) {
  if (rows == 0) return SPECVLM_OK;
  argmax_rows_kernel<<<rows, kArgmaxThreads, 0, stream>>>(logits, V, row_stride, out);
  return check_cuda(cudaGetLastError(), "argmax launch");
}

}  // namespace specvlm

extern "C" int specvlm_argmax(const float* target_logits, int B, int T, int V, int64_t row_stride,
                              int32_t* argmax_tokens, void* stream) {
  SPECVLM_REQUIRE(B >= 0 && T >= 1 && T <= SPECVLM_MAX_TREE, "argmax: need B >= 0 and 1 <= T <= 64");
  SPECVLM_REQUIRE(V >= 1, "argmax: V must be positive");
  if (B == 0) return SPECVLM_OK;
  SPECVLM_REQUIRE(target_logits != nullptr && argmax_tokens != nullptr, "argmax: null pointer");
  SPECVLM_REQUIRE(row_stride >= V && (row_stride & 3) == 0, "argmax: row_stride must be >= V and a multiple of 4");
  SPECVLM_REQUIRE(specvlm::aligned16(target_logits), "argmax: target_logits must be 16-byte aligned");
  return specvlm::launch_argmax(target_logits, B * T, V, row_stride, argmax_tokens,
                                static_cast<cudaStream_t>(stream));
}
