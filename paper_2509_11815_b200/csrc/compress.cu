// Parameter-free visual token compression (Section 3.4: the elastic compressor's pruning, which
// drops tokens at random, and pooling). Pooling: 1-D average over windows of `ratio` consecutive
// visual tokens (the last window takes what remains), fp32 accumulation, bf16 in and out.
// Pruning: the kept rows, given by index, are copied bit for bit. Both are plain HBM streams with
// 16-byte accesses.
#include "common.cuh"

#include <cuda_bf16.h>

namespace specvlm {

__device__ __forceinline__ void add8(float (&acc)[8], const uint4& u) {
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float2 f = __bfloat1622float2(h[j]);
    acc[2 * j] += f.x;
    acc[2 * j + 1] += f.y;
  }
}

__global__ void visual_pool_kernel(const uint16_t* __restrict__ x, int N, int C8, int ratio, int M,
                                   uint16_t* __restrict__ y) {
  const int m = blockIdx.x, b = blockIdx.y;
  const int n0 = m * ratio, n1 = min(n0 + ratio, N);
  const float inv = 1.0f / static_cast<float>(n1 - n0);
  const uint4* src = reinterpret_cast<const uint4*>(x) + (static_cast<int64_t>(b) * N + n0) * C8;
  uint4* dst = reinterpret_cast<uint4*>(y) + (static_cast<int64_t>(b) * M + m) * C8;
  for (int c = threadIdx.x; c < C8; c += blockDim.x) {
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int n = 0; n < n1 - n0; ++n) add8(acc, src[static_cast<int64_t>(n) * C8 + c]);
    uint4 out;
    __nv_bfloat162* o = reinterpret_cast<__nv_bfloat162*>(&out);
#pragma unroll
    for (int j = 0; j < 4; ++j) o[j] = __floats2bfloat162_rn(acc[2 * j] * inv, acc[2 * j + 1] * inv);
    dst[c] = out;
  }
}

__global__ void visual_prune_kernel(const uint16_t* __restrict__ x, const int32_t* __restrict__ keep, int N, int C8,
                                    int M, uint16_t* __restrict__ y, int32_t* __restrict__ status) {
  const int m = blockIdx.x, b = blockIdx.y;
  const int n = keep[b * M + m];
  const bool ok = n >= 0 && n < N;
  if (!ok && threadIdx.x == 0 && status != nullptr) atomicOr(status, SPECVLM_STATUS_BAD_ACCEPT);
  const uint4* src = reinterpret_cast<const uint4*>(x) + (static_cast<int64_t>(b) * N + (ok ? n : 0)) * C8;
  uint4* dst = reinterpret_cast<uint4*>(y) + (static_cast<int64_t>(b) * M + m) * C8;
  for (int c = threadIdx.x; c < C8; c += blockDim.x) dst[c] = ok ? src[c] : make_uint4(0, 0, 0, 0);
}

}  // namespace specvlm

using namespace specvlm;

extern "C" int specvlm_visual_pool(const uint16_t* x, int B, int N, int C, int ratio, uint16_t* y, void* stream) {
  SPECVLM_REQUIRE(B >= 0 && B <= 65535 && N >= 1 && C >= 8 && (C % 8) == 0, "visual_pool: need N >= 1 and C a positive multiple of 8");
  SPECVLM_REQUIRE(ratio >= 1, "visual_pool: ratio must be >= 1");
  if (B == 0) return SPECVLM_OK;
  SPECVLM_REQUIRE(x && y && aligned16(x) && aligned16(y), "visual_pool: null or misaligned pointer");
  const int M = (N + ratio - 1) / ratio;
  visual_pool_kernel<<<dim3(M, B), 256, 0, static_cast<cudaStream_t>(stream)>>>(x, N, C / 8, ratio, M, y);
  return check_cuda(cudaGetLastError(), "visual_pool launch");
}

extern "C" int specvlm_visual_prune(const uint16_t* x, const int32_t* keep_idx, int B, int N, int C, int M,
                                    uint16_t* y, int32_t* status, void* stream) {
  SPECVLM_REQUIRE(B >= 0 && B <= 65535 && N >= 1 && M >= 0 && C >= 8 && (C % 8) == 0, "visual_prune: bad shape");
  if (B == 0 || M == 0) return SPECVLM_OK;
  SPECVLM_REQUIRE(x && y && keep_idx && aligned16(x) && aligned16(y), "visual_prune: null or misaligned pointer");
  visual_prune_kernel<<<dim3(M, B), 256, 0, static_cast<cudaStream_t>(stream)>>>(x, keep_idx, N, C / 8, M, y, status);
  return check_cuda(cudaGetLastError(), "visual_prune launch");
}
