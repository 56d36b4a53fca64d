// Draft-tree construction primitives (Section 4.1: EAGLE-2 style tree, top-k 10 expansion,
// 60 tokens). The draft model itself is out of scope; these are the two tree-building steps
// around it: (1) the k most probable next tokens of an expanded node with their
// log-probabilities, (2) the final rerank of all candidates by cumulative score into a tree
// with parent < child labels, its mask words, depths and position ids.
#include "common.cuh"

#include <limits.h>
#include <math.h>

namespace specvlm {

constexpr int kTopkThreads = 512;
constexpr int kMaxK = 16;

struct Cand {
  float v;
  int i;
};
// larger value first; equal values: lower index first
__device__ __forceinline__ bool before(const Cand& a, const Cand& b) { return a.v > b.v || (a.v == b.v && a.i < b.i); }

// One block per logits row. Every thread first loads its strided share of the row into registers
// (up to 64 values, i.e. rows of up to 32768 entries; longer rows re-read global memory) and
// accumulates an online (max, sum) for the row's log-sum-exp. Then k rounds: each thread finds its
// best value that comes strictly after the previous round's winner in (value descending, index
// ascending) order, and a block-wide reduction picks the round's winner.
constexpr int kTopkRegs = 64;

__global__ void __launch_bounds__(kTopkThreads)
topk_logprob_kernel(const float* __restrict__ logits, int V, int64_t row_stride, int k,
                    int32_t* __restrict__ tokens, float* __restrict__ logprob) {
  const int row = blockIdx.x;
  const float* x = logits + static_cast<int64_t>(row) * row_stride;
  __shared__ float s_m[kTopkThreads / 32], s_z[kTopkThreads / 32];
  __shared__ Cand s_c[kTopkThreads / 32];
  __shared__ float s_lse;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const bool in_regs = V <= kTopkRegs * kTopkThreads;
  float vals[kTopkRegs];
  float m = -INFINITY, z = 0.f;
#pragma unroll
  for (int u = 0; u < kTopkRegs; ++u) {
    const int v = threadIdx.x + u * kTopkThreads;
    vals[u] = (in_regs && v < V) ? x[v] : -INFINITY;
  }
  if (in_regs) {
#pragma unroll
    for (int u = 0; u < kTopkRegs; ++u) m = fmaxf(m, vals[u]);
#pragma unroll
    for (int u = 0; u < kTopkRegs; ++u) z += (vals[u] == -INFINITY) ? 0.f : __expf(vals[u] - m);
  } else {
    for (int v = threadIdx.x; v < V; v += kTopkThreads) {
      const float val = x[v];
      if (val > m) { z = z * __expf(m - val) + 1.f; m = val; } else { z += __expf(val - m); }
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, m, off), oz = __shfl_xor_sync(0xffffffffu, z, off);
    const float nm = fmaxf(m, om);
    z = (m == -INFINITY ? 0.f : z * __expf(m - nm)) + (om == -INFINITY ? 0.f : oz * __expf(om - nm));
    m = nm;
  }
  if (lane == 0) { s_m[warp] = m; s_z[warp] = z; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float gm = -INFINITY, gz = 0.f;
    for (int q = 0; q < kTopkThreads / 32; ++q) {
      const float nm = fmaxf(gm, s_m[q]);
      gz = (gm == -INFINITY ? 0.f : gz * __expf(gm - nm)) + (s_m[q] == -INFINITY ? 0.f : s_z[q] * __expf(s_m[q] - nm));
      gm = nm;
    }
    s_lse = gm + logf(gz);
  }
  Cand last{INFINITY, -1};  // everything comes after it
  for (int r = 0; r < k; ++r) {
    Cand c{-INFINITY, INT_MAX};
    if (in_regs) {
      // within a thread indices grow with u, so the first maximum in u order has the lowest index
#pragma unroll
      for (int u = 0; u < kTopkRegs; ++u) {
        const int v = threadIdx.x + u * kTopkThreads;
        const float val = vals[u];
        const bool after = val < last.v || (val == last.v && v > last.i);
        if (after && val > c.v && v < V) c = Cand{val, v};
      }
    } else {
      for (int v = threadIdx.x; v < V; v += kTopkThreads) {
        const Cand e{x[v], v};
        if (before(last, e) && before(e, c)) c = e;
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      Cand o{__shfl_xor_sync(0xffffffffu, c.v, off), __shfl_xor_sync(0xffffffffu, c.i, off)};
      if (before(o, c)) c = o;
    }
    __syncthreads();  // s_c of the previous round (and s_lse) settled
    if (lane == 0) s_c[warp] = c;
    __syncthreads();
    Cand w = s_c[0];
#pragma unroll
    for (int q = 1; q < kTopkThreads / 32; ++q)
      if (before(s_c[q], w)) w = s_c[q];
    last = w;
    if (threadIdx.x == 0) {
      tokens[static_cast<int64_t>(row) * k + r] = (w.i == INT_MAX) ? 0 : w.i;
      logprob[static_cast<int64_t>(row) * k + r] = w.v - s_lse;
    }
  }
}

constexpr int kRerankThreads = 1024;  // also the candidate limit

// One block per sequence, one thread per candidate. Ranks come from counting: candidate i is
// kept iff fewer than T-1 other candidates come before it in (score descending, index) order;
// its new label is the number of kept candidates before it in (depth, score descending, index).
__global__ void __launch_bounds__(kRerankThreads)
tree_rerank_kernel(const int32_t* __restrict__ cand_parent, const float* __restrict__ cand_score,
                   const int32_t* __restrict__ cand_token, const int32_t* __restrict__ prefix_len, int C, int T,
                   int32_t* __restrict__ tree_parent, int32_t* __restrict__ draft_tokens, int32_t* __restrict__ kept_out,
                   uint64_t* __restrict__ mask_bits, int32_t* __restrict__ depth_out, int32_t* __restrict__ pos_out,
                   int32_t* __restrict__ status) {
  const int b = blockIdx.x, i = threadIdx.x;
  cand_parent += static_cast<int64_t>(b) * C; cand_score += static_cast<int64_t>(b) * C;
  cand_token += static_cast<int64_t>(b) * C;
  __shared__ __align__(16) float s_score[kRerankThreads];
  __shared__ short s_par[kRerankThreads], s_depth[kRerankThreads], s_label[kRerankThreads];
  __shared__ int s_bad;
  __shared__ int s_tpar[SPECVLM_MAX_TREE];
  if (i == 0) s_bad = 0;
  s_score[i] = (i < C) ? cand_score[i] : -INFINITY;
  if (i < C) {
    const int p = cand_parent[i];
    s_par[i] = static_cast<short>(p);
    s_label[i] = -1;
  }
  __syncthreads();
  bool keep = false;
  int depth = 0;
  if (i < C) {
    const int p = s_par[i];
    if ((i == 0) ? (p != -1) : (p < 0 || p >= i)) s_bad = 1;
  }
  __syncthreads();
  const bool bad = s_bad != 0;
  if (i < C && !bad) {
    int n = i;
    while (n > 0) { n = s_par[n]; ++depth; }
    s_depth[i] = static_cast<short>(depth);
    if (i == 0) {
      keep = true;
    } else {
      const float si = s_score[i];
      int rank = 0;
      // four scores per shared-memory load; entries at or beyond C were filled with -inf
      const float4* sc4 = reinterpret_cast<const float4*>(s_score);
      for (int j4 = 0; j4 < (C + 3) / 4; ++j4) {
        const float4 sj = sc4[j4];
        const int j = 4 * j4;
        rank += (j > 0 && (sj.x > si || (sj.x == si && j < i))) ? 1 : 0;
        rank += (sj.y > si || (sj.y == si && j + 1 < i)) ? 1 : 0;
        rank += (sj.z > si || (sj.z == si && j + 2 < i)) ? 1 : 0;
        rank += (sj.w > si || (sj.w == si && j + 3 < i)) ? 1 : 0;
      }
      keep = rank < T - 1;
    }
    s_label[i] = keep ? 0 : -1;
  }
  __syncthreads();
  // compact list of the kept candidates, so that the relabelling only compares kept ones
  __shared__ int s_nkept;
  __shared__ short s_kept[SPECVLM_MAX_TREE];
  if (i == 0) s_nkept = 0;
  __syncthreads();
  if (keep) {
    const int slot = atomicAdd(&s_nkept, 1);
    if (slot < SPECVLM_MAX_TREE) s_kept[slot] = static_cast<short>(i);
  }
  __syncthreads();
  int label = -1;
  if (keep) {
    const float si = s_score[i];
    const int nk = min(s_nkept, SPECVLM_MAX_TREE);
    int cnt = 0;
    for (int q = 0; q < nk; ++q) {
      const int j = s_kept[q];
      if (j == i) continue;
      const int dj = s_depth[j];
      const float sj = s_score[j];
      const bool first = (dj < depth) || (dj == depth && (sj > si || (sj == si && j < i)));
      cnt += first ? 1 : 0;
    }
    label = cnt;
  }
  __syncthreads();
  if (keep) s_label[i] = static_cast<short>(label);
  __syncthreads();
  if (keep) {
    const int pl = (i == 0) ? -1 : s_label[s_par[i]];
    if (i > 0 && pl < 0) s_bad = 1;  // parent not kept: scores increased along a path
    const int64_t o = static_cast<int64_t>(b) * T + label;
    tree_parent[o] = pl;
    draft_tokens[o] = cand_token[i];
    if (kept_out != nullptr) kept_out[o] = i;
    if (depth_out != nullptr) depth_out[o] = depth;
    if (pos_out != nullptr) pos_out[o] = (prefix_len != nullptr ? prefix_len[b] : 0) + depth;
    s_tpar[label] = pl;
  }
  __syncthreads();
  if (i < T && mask_bits != nullptr && !bad && s_bad == 0) {
    uint64_t bits = 0;
    int n = i;
    for (int step = 0; step < SPECVLM_MAX_TREE && n >= 0; ++step) { bits |= 1ull << n; n = s_tpar[n]; }
    mask_bits[static_cast<int64_t>(b) * T + i] = bits;
  }
  if (i == 0 && s_bad != 0 && status != nullptr) atomicOr(status, SPECVLM_STATUS_BAD_TREE);
}

}  // namespace specvlm

using namespace specvlm;

extern "C" int specvlm_topk_logprob(const float* logits, int rows, int V, int64_t row_stride, int k,
                                    int32_t* tokens, float* logprob, void* stream) {
  SPECVLM_REQUIRE(rows >= 0 && V >= 1, "topk_logprob: bad shape");
  SPECVLM_REQUIRE(k >= 1 && k <= kMaxK && k <= V, "topk_logprob: need 1 <= k <= 16 and k <= V");
  if (rows == 0) return SPECVLM_OK;
  SPECVLM_REQUIRE(logits && tokens && logprob, "topk_logprob: null pointer");
  SPECVLM_REQUIRE(row_stride >= V, "topk_logprob: row_stride must be >= V");
  topk_logprob_kernel<<<rows, kTopkThreads, 0, static_cast<cudaStream_t>(stream)>>>(logits, V, row_stride, k,
                                                                                        tokens, logprob);
  return check_cuda(cudaGetLastError(), "topk_logprob launch");
}

extern "C" int specvlm_tree_rerank(const int32_t* cand_parent, const float* cand_score, const int32_t* cand_token,
                                   const int32_t* prefix_len, int B, int C, int T, int32_t* tree_parent,
                                   int32_t* draft_tokens, int32_t* kept_candidates, uint64_t* mask_bits,
                                   int32_t* depth, int32_t* pos, int32_t* status, void* stream) {
  SPECVLM_REQUIRE(B >= 0 && T >= 1 && T <= SPECVLM_MAX_TREE, "tree_rerank: need B >= 0 and 1 <= T <= 64");
  SPECVLM_REQUIRE(C >= T && C <= kRerankThreads, "tree_rerank: need T <= C <= 1024 candidates");
  if (B == 0) return SPECVLM_OK;
  SPECVLM_REQUIRE(cand_parent && cand_score && cand_token && tree_parent && draft_tokens, "tree_rerank: null pointer");
  SPECVLM_REQUIRE(pos == nullptr || prefix_len != nullptr, "tree_rerank: pos needs prefix_len");
  tree_rerank_kernel<<<B, kRerankThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      cand_parent, cand_score, cand_token, prefix_len, C, T, tree_parent, draft_tokens, kept_candidates, mask_bits,
      depth, pos, status);
  return check_cuda(cudaGetLastError(), "tree_rerank launch");
}
