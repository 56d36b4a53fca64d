// Temperature > 0 acceptance on the draft tree by speculative sampling (Section 3.1: speculative
// sampling discards incorrect tokens; Section 4.1: stochastic decoding at temperature 1 is
// evaluated and the target distribution is preserved).
//
// Rule (children are fixed candidates, tried in index order): at the current node with
// p = softmax(logits / temperature), child c with token x is kept with probability
// p(x) / (1 - mass already rejected); a rejected token is removed from p. If a child is kept the
// walk descends; otherwise the next token is drawn from what is left of p by inverse CDF. All
// random numbers are inputs (one per node for its keep test, one per node for the draw there).
//
// One block of 1024 threads per sequence. Per visited node: block-wide max and sum of
// exp((l - max) / temperature) over the vocabulary row (fp32, fixed reduction order), the
// sequential child loop on thread 0, and, when the walk stops, an inverse-CDF search: every
// thread sums a contiguous chunk of the row (removed tokens skipped), the chunk sums are
// scanned, and the thread whose chunk contains the target walks it element by element.
#include "common.cuh"

#include <math.h>

namespace specvlm {

constexpr int kSampleThreads = 1024;
constexpr int kMaxChildren = SPECVLM_MAX_TREE;

__device__ __forceinline__ float block_reduce(float v, bool is_max, float* s_red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float o = __shfl_xor_sync(0xffffffffu, v, off);
    v = is_max ? fmaxf(v, o) : v + o;
  }
  __syncthreads();  // s_red may still be read from the previous call
  if (lane == 0) s_red[warp] = v;
  __syncthreads();
  float r = s_red[lane];  // kSampleThreads / 32 == 32 partials
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float o = __shfl_xor_sync(0xffffffffu, r, off);
    r = is_max ? fmaxf(r, o) : r + o;
  }
  return r;
}

__global__ void __launch_bounds__(kSampleThreads)
accept_sample_kernel(const int32_t* __restrict__ draft, const int32_t* __restrict__ parent,
                     const float* __restrict__ logits, const float* __restrict__ u_accept,
                     const float* __restrict__ u_sample, float inv_temp, int T, int V,
                     int32_t* __restrict__ accepted_idx, int acc_stride, int32_t* __restrict__ accept_len,
                     int32_t* __restrict__ next_token, int32_t* __restrict__ status) {
  const int b = blockIdx.x;
  draft += b * T; parent += b * T; u_accept += b * T; u_sample += b * T;
  logits += static_cast<int64_t>(b) * T * V;
  __shared__ int s_parent[SPECVLM_MAX_TREE], s_draft[SPECVLM_MAX_TREE], s_path[SPECVLM_MAX_TREE];
  __shared__ int s_gone[kMaxChildren];
  __shared__ float s_red[32], s_chunk[kSampleThreads];
  __shared__ int s_next, s_ngone, s_bad, s_result;
  if (threadIdx.x == 0) s_bad = 0;
  __syncthreads();
  if (threadIdx.x < T) {
    const int pr = parent[threadIdx.x];
    s_parent[threadIdx.x] = pr;
    s_draft[threadIdx.x] = draft[threadIdx.x];
    if ((threadIdx.x == 0) ? (pr != -1) : (pr < 0 || pr >= static_cast<int>(threadIdx.x))) s_bad = 1;
  }
  __syncthreads();
  const bool bad_tree = s_bad != 0;
  int cur = 0, depth = 0;
  if (threadIdx.x == 0) s_path[0] = 0;

  for (int guard = 0; guard < SPECVLM_MAX_TREE; ++guard) {
    const float* row = logits + static_cast<int64_t>(cur) * V;
    float m = -INFINITY;
    for (int v = threadIdx.x; v < V; v += kSampleThreads) m = fmaxf(m, row[v]);
    m = block_reduce(m, true, s_red);
    float z = 0.f;
    for (int v = threadIdx.x; v < V; v += kSampleThreads) z += __expf((row[v] - m) * inv_temp);
    z = block_reduce(z, false, s_red);

    if (threadIdx.x == 0) {
      float removed = 0.f;
      int ngone = 0, kept = -1;
      if (!bad_tree) {
        for (int c = cur + 1; c < T; ++c) {
          if (s_parent[c] != cur) continue;
          const int x = s_draft[c];
          bool gone = x < 0 || x >= V;
          for (int j = 0; j < ngone; ++j) gone = gone || (s_gone[j] == x);
          const float px = gone ? 0.f : __expf((row[x] - m) * inv_temp) / z;
          const float rest = 1.f - removed;
          if (rest > 0.f && u_accept[c] < px / rest) { kept = c; break; }
          removed += px;
          if (!gone && ngone < kMaxChildren) s_gone[ngone++] = x;
        }
      }
      s_next = kept;
      s_ngone = ngone;
    }
    __syncthreads();
    const int kept = s_next;
    if (kept >= 0) {
      cur = kept;
      ++depth;
      if (threadIdx.x == 0) s_path[depth] = kept;
      __syncthreads();
      continue;
    }
    // ---- draw the next token from what is left of p: first v with cumulative weight > target
    const int ngone = s_ngone;
    const int chunk = (V + kSampleThreads - 1) / kSampleThreads;
    const int v0 = threadIdx.x * chunk, v1 = min(v0 + chunk, V);
    float local = 0.f;
    for (int v = v0; v < v1; ++v) {
      bool gone = false;
      for (int j = 0; j < ngone; ++j) gone = gone || (s_gone[j] == v);
      if (!gone) local += __expf((row[v] - m) * inv_temp);
    }
    s_chunk[threadIdx.x] = local;
    if (threadIdx.x == 0) s_result = -1;
    __syncthreads();
    if (threadIdx.x < 32) {
      // warp 0 scans the 1024 chunk sums: 32 per lane, then across lanes
      float run = 0.f;
      for (int j = 0; j < 32; ++j) run += s_chunk[threadIdx.x * 32 + j];
      float incl = run;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const float o = __shfl_up_sync(0xffffffffu, incl, off);
        if (static_cast<int>(threadIdx.x) >= off) incl += o;
      }
      const float total = __shfl_sync(0xffffffffu, incl, 31);
      const float target = u_sample[cur] * total;
      float before = incl - run;  // weight of all chunks owned by lower lanes
      // the lane whose span [before, incl) contains the target walks its 32 chunks, then the chunk
      const bool mine = (target >= before && target < incl) || (threadIdx.x == 31 && target >= incl);
      if (mine) {
        int res = -1;
        for (int j = 0; j < 32 && res < 0; ++j) {
          const int t2 = threadIdx.x * 32 + j;
          const float cs = s_chunk[t2];
          if (target < before + cs || (threadIdx.x == 31 && j == 31)) {
            float acc = before;
            const int a0 = t2 * chunk, a1 = min(a0 + chunk, V);
            for (int v = a0; v < a1; ++v) {
              bool gone = false;
              for (int q = 0; q < ngone; ++q) gone = gone || (s_gone[q] == v);
              if (gone) continue;
              acc += __expf((row[v] - m) * inv_temp);
              res = v;  // last candidate that is still present
              if (acc > target) break;
            }
            if (res < 0) before += cs;  // empty chunk (all removed / out of range): keep looking
          } else {
            before += cs;
          }
        }
        if (res < 0) {  // numerical corner: fall back to the last token that is still present
          for (int v = V - 1; v >= 0 && res < 0; --v) {
            bool gone = false;
            for (int q = 0; q < ngone; ++q) gone = gone || (s_gone[q] == v);
            if (!gone) res = v;
          }
        }
        s_result = res;
      }
    }
    __syncthreads();
    break;
  }
  for (int j = threadIdx.x; j < acc_stride; j += kSampleThreads)
    accepted_idx[static_cast<int64_t>(b) * acc_stride + j] = (j <= depth) ? s_path[j] : -1;
  if (threadIdx.x == 0) {
    accept_len[b] = depth;
    next_token[b] = s_result;
    if (bad_tree && status != nullptr) atomicOr(status, SPECVLM_STATUS_BAD_TREE);
  }
}

}  // namespace specvlm

using namespace specvlm;

extern "C" int specvlm_accept_sample(const int32_t* draft_tokens, const int32_t* tree_parent,
                                     const float* target_logits, const float* uniforms_accept,
                                     const float* uniforms_sample, float temperature, int B, int T, int V,
                                     int32_t* accepted_idx, int acc_stride, int32_t* accept_len,
                                     int32_t* next_token, int32_t* status, void* stream) {
  SPECVLM_REQUIRE(B >= 0 && T >= 1 && T <= SPECVLM_MAX_TREE, "accept_sample: need B >= 0 and 1 <= T <= 64");
  SPECVLM_REQUIRE(V >= 1, "accept_sample: V must be positive");
  SPECVLM_REQUIRE(temperature > 0.f && isfinite(temperature), "accept_sample: temperature must be positive (use specvlm_accept for 0)");
  if (B == 0) return SPECVLM_OK;
  SPECVLM_REQUIRE(draft_tokens && tree_parent && target_logits && uniforms_accept && uniforms_sample &&
                      accepted_idx && accept_len && next_token,
                  "accept_sample: null pointer");
  SPECVLM_REQUIRE(acc_stride >= 1, "accept_sample: acc_stride must be >= 1");
  accept_sample_kernel<<<B, kSampleThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      draft_tokens, tree_parent, target_logits, uniforms_accept, uniforms_sample, 1.0f / temperature, T, V,
      accepted_idx, acc_stride, accept_len, next_token, status);
  return check_cuda(cudaGetLastError(), "accept_sample launch");
}
