// Vocabulary-wide argmax of the target logits at every tree node (the greedy target
// token used by temperature-0 verification; part of the sampling cost of Eq. 1).
//
// One cluster of four thread blocks per logits row. Every thread keeps the (value, lowest
// index) of the maximum among the float4 groups it streams (128-bit coalesced loads), then
// the pairs are reduced with "greater value, else lower index", which reproduces a
// sequential scan with strict '>' bit for bit. HBM-bound: V * 4 bytes per row, read once.
#include "common.cuh"

#include <cooperative_groups.h>
#include <limits.h>

namespace specvlm {

constexpr int kArgmaxThreads = 256;
constexpr int kArgmaxSplit = 4;  // CTAs per row = cluster size

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

// One cluster of kArgmaxSplit CTAs per logits row; each CTA scans a contiguous quarter of the
// row's float4 groups, the partial (value, index) pairs meet in the first CTA's shared memory
// through distributed shared memory.
__global__ void __launch_bounds__(kArgmaxThreads)
argmax_rows_kernel(const float* __restrict__ logits, int V, int64_t row_stride,
                   int32_t* __restrict__ out) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  const int row = blockIdx.x / kArgmaxSplit;
  const int part = blockIdx.x % kArgmaxSplit;  // == rank in the cluster
  const float* x = logits + static_cast<int64_t>(row) * row_stride;
  const float4* x4 = reinterpret_cast<const float4*>(x);
  const int n4 = V >> 2;
  const int per = (n4 + kArgmaxSplit - 1) / kArgmaxSplit;
  const int g0 = part * per, g1 = min(g0 + per, n4);

  grid_dependency_sync();
  cluster.barrier_arrive();  // matched by the wait below: every CTA of the cluster has started by then
  Best best{-INFINITY, INT_MAX};
  // -inf never passes '>' against the initial -inf; INT_MAX then loses every index tie,
  // and an all -inf row ends as index 0 below.
  int g = g0 + threadIdx.x;
  // Eight independent 16-byte loads in flight per thread per trip (a 32000-entry row is one trip).
  for (; g < g1; g += 8 * kArgmaxThreads) {
    float4 a[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int gu = g + u * kArgmaxThreads;
      a[u] = (gu < g1) ? __ldcs(x4 + gu) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = (g + u * kArgmaxThreads) * 4;
      take(best, a[u].x, i); take(best, a[u].y, i + 1); take(best, a[u].z, i + 2); take(best, a[u].w, i + 3);
    }
  }
  if (part == kArgmaxSplit - 1)  // the row's scalar tail belongs to the last part
    for (int i = (n4 << 2) + threadIdx.x; i < V; i += kArgmaxThreads) take(best, x[i], i);

#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    Best o{__shfl_xor_sync(0xffffffffu, best.v, off), __shfl_xor_sync(0xffffffffu, best.i, off)};
    best = better(best, o);
  }
  constexpr int kWarps = kArgmaxThreads / 32;
  __shared__ float sv[kArgmaxSplit * kWarps];
  __shared__ int si[kArgmaxSplit * kWarps];
  cluster.barrier_wait();
  if ((threadIdx.x & 31) == 0) {
    // every CTA deposits its warps' results in the first CTA's arrays
    float* dv = cluster.map_shared_rank(sv, 0);
    int* di = cluster.map_shared_rank(si, 0);
    dv[part * kWarps + (threadIdx.x >> 5)] = best.v;
    di[part * kWarps + (threadIdx.x >> 5)] = best.i;
  }
  cluster.sync();
  if (part == 0 && threadIdx.x < 32) {
    Best b{-INFINITY, INT_MAX};
    if (threadIdx.x < kArgmaxSplit * kWarps) b = Best{sv[threadIdx.x], si[threadIdx.x]};
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
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(kArgmaxSplit) * rows);  // rows along x: no 65535 limit
  cfg.blockDim = dim3(kArgmaxThreads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kArgmaxSplit;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // the kernel starts with grid_dependency_sync()
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return check_cuda(cudaLaunchKernelEx(&cfg, argmax_rows_kernel, logits, V, row_stride, out), "argmax launch");
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
