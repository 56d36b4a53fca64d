// Draft-tree construction primitives (Section 4.1: EAGLE-2 style tree, top-k 10 expansion,
// 60 tokens). The draft model itself is out of scope; these are the two tree-building steps
// around it: (1) the k most probable next tokens of an expanded node with their
// log-probabilities, (2) the final rerank of all candidates by cumulative score into a tree
// with parent < child labels, its mask words, depths and position ids.
#include "common.cuh"

#include <cooperative_groups.h>
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
      if (val > m) { z = z * __expf(m - val) + 1.f; m = val; } else if (val > -INFINITY) { z += __expf(val - m); }
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

// ---- cluster version: the row is shared by eight thread blocks
//
// One cluster of kTkSplit blocks per logits row. Every thread keeps kU groups of four consecutive
// logits in registers (one 16-byte load each, all in flight together). Each block computes the
// (max, sum) pair and the sorted top k of its share with k selection rounds over registers; the
// lists and pairs meet in the first block's shared memory through distributed shared memory,
// where the final order is found by counting: a candidate's position is the number of candidates
// that come before it in (value descending, index ascending) order.
constexpr int kTkThreads = 256;
constexpr int kTkSplit = 8;

// Unsigned key whose integer order is the order of the floats (-0 counted as +0).
__device__ __forceinline__ unsigned ordered_key(float v) {
  const unsigned u = __float_as_uint(v + 0.f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_value(unsigned key) {
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// Entries of exhausted lists carry value -inf and an index at or above kSentinel0, made unique
// by the writer, so that (value descending, index ascending) orders all entries strictly.
constexpr int kSentinel0 = INT_MAX - 4096;

// Position of entry `me` among kLists sorted lists of k entries stored kMaxK apart: the number of
// entries that come before it = the sum of its lower bounds in every list (its own place in its
// own list). The binary searches of different lists are independent of one another.
template <int kLists>
__device__ __forceinline__ int rank_among(const Cand* lists, int k, const Cand me) {
  int rank = 0;
#pragma unroll
  for (int l = 0; l < kLists; ++l) {
    int lo = 0, hi = k;
#pragma unroll
    for (int step = 0; step < 5; ++step) {  // k <= 16 < 2^5
      if (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (before(lists[l * kMaxK + mid], me)) lo = mid + 1; else hi = mid;
      }
    }
    rank += lo;
  }
  return rank;
}

template <int kU>
__global__ void __launch_bounds__(kTkThreads)
topk_cluster_kernel(const float* __restrict__ logits, int V, int64_t row_stride, int k, int vec,
                    int32_t* __restrict__ tokens, float* __restrict__ logprob) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  const int row = blockIdx.x / kTkSplit, part = blockIdx.x % kTkSplit;  // part == rank in the cluster
  const float* x = logits + static_cast<int64_t>(row) * row_stride;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  constexpr int kWarps = kTkThreads / 32;
  __shared__ float s_m[kWarps], s_z[kWarps];
  __shared__ Cand s_all[kTkSplit * kMaxK];  // used in the first block: every block's sorted list
  __shared__ float s_pm[kTkSplit], s_pz[kTkSplit];
  cluster.barrier_arrive();  // matched by the wait before the first remote store

  const int n4 = (V + 3) >> 2;
  const int per = (n4 + kTkSplit - 1) / kTkSplit;  // host guarantees per <= kU * kTkThreads
  const int g0 = part * per, g1 = min(g0 + per, n4);
  float vals[kU * 4];
#pragma unroll
  for (int u = 0; u < kU; ++u) {
    const int g = g0 + u * kTkThreads + threadIdx.x;
    float4 t = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    if (g < g1) {
      if (vec) {
        t = __ldg(reinterpret_cast<const float4*>(x) + g);
      } else {
        const int v = g << 2;
        t.x = x[v];
        if (v + 1 < V) t.y = x[v + 1];
        if (v + 2 < V) t.z = x[v + 2];
        if (v + 3 < V) t.w = x[v + 3];
      }
    }
    vals[4 * u] = t.x; vals[4 * u + 1] = t.y; vals[4 * u + 2] = t.z; vals[4 * u + 3] = t.w;
  }
  // element e of group u is logit index 4 * (g0 + u * kTkThreads + threadIdx.x) + e: increasing in (u, e)
  const int vbase = (g0 + static_cast<int>(threadIdx.x)) << 2;

  float m = -INFINITY, z = 0.f;
#pragma unroll
  for (int i = 0; i < kU * 4; ++i) m = fmaxf(m, vals[i]);
#pragma unroll
  for (int i = 0; i < kU * 4; ++i) z += (vals[i] == -INFINITY) ? 0.f : __expf(vals[i] - m);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, m, off), oz = __shfl_xor_sync(0xffffffffu, z, off);
    const float nm = fmaxf(m, om);
    z = (m == -INFINITY ? 0.f : z * __expf(m - nm)) + (om == -INFINITY ? 0.f : oz * __expf(om - nm));
    m = nm;
  }
  if (lane == 0) { s_m[warp] = m; s_z[warp] = z; }

  // ---- every warp finds the sorted top k of its own share, no block-wide step.
  // Prefilter: the k-th best of the 32 lanes' own best entries (k rounds over one value per lane)
  // is a threshold that at least k entries of the warp reach, so the warp's top k are among the
  // entries that are not after it; typically fewer than 2 k entries pass. They are compacted into
  // a short list with ballots and ranked by counting. If more than kListCap pass (a lane holding
  // many of the warp's largest values), the warp falls back to k selection rounds over all of its
  // registers.
  constexpr int kListCap = 64;
  __shared__ Cand s_list[kWarps][kListCap];
  __shared__ Cand s_wl[kWarps * kMaxK];  // every warp's sorted top k
  Cand kept{-INFINITY, INT_MAX};
  Cand lm{-INFINITY, INT_MAX};  // this lane's best entry: first maximum in (u, e) order = lowest index
#pragma unroll
  for (int u = 0; u < kU; ++u) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float val = vals[4 * u + e];
      if (val > lm.v) lm = Cand{val, vbase + u * (kTkThreads * 4) + e};
    }
  }
  Cand thr{-INFINITY, INT_MAX};
  {
    const unsigned lkey = ordered_key(lm.v);
    bool used = false;
    for (int r = 0; r < k; ++r) {
      const unsigned key = used ? 0u : lkey;  // every real key is above 0
      const unsigned kmax = __reduce_max_sync(0xffffffffu, key);
      const unsigned imin =
          __reduce_min_sync(0xffffffffu, (!used && key == kmax) ? static_cast<unsigned>(lm.i) : 0xffffffffu);
      if (!used && key == kmax && static_cast<unsigned>(lm.i) == imin) used = true;
      thr = Cand{key_value(kmax), static_cast<int>(imin)};
    }
    // lanes without any selectable entry report (-inf, INT_MAX): then every selectable entry passes
    if (thr.i == INT_MAX || !(thr.v > -INFINITY)) thr = Cand{-INFINITY, INT_MAX};
  }
  int n_list = 0;  // warp-uniform
#pragma unroll
  for (int u = 0; u < kU; ++u) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int v = vbase + u * (kTkThreads * 4) + e;
      const float val = vals[4 * u + e];
      const bool pass = val > -INFINITY && (val > thr.v || (val == thr.v && v <= thr.i));
      const unsigned ball = __ballot_sync(0xffffffffu, pass);
      if (ball != 0u) {
        const int slot = n_list + __popc(ball & ((1u << lane) - 1u));
        if (pass && slot < kListCap) s_list[warp][slot] = Cand{val, v};
        n_list += __popc(ball);
      }
    }
  }
  __syncwarp();
  if (n_list <= kListCap) {
    // rank by counting inside the list; places n_list .. k-1 (fewer than k selectable entries) stay empty
    for (int q = lane; q < n_list; q += 32) {
      const Cand me = s_list[warp][q];
      int rank = 0;
      for (int o = 0; o < n_list; ++o) rank += before(s_list[warp][o], me) ? 1 : 0;
      if (rank < k) s_wl[warp * kMaxK + rank] = me;
    }
    // fewer than k selectable entries: the remaining places get sentinels, unique per entry
    if (lane >= n_list && lane < k)
      s_wl[warp * kMaxK + lane] = Cand{-INFINITY, kSentinel0 + (part * kWarps + warp) * kMaxK + lane};
  } else {
    // k selection rounds: each round's winner is the best entry that comes strictly after the
    // previous winner, found with two warp-wide integer reductions; lane r keeps round r's winner
    Cand last{INFINITY, -1};
    for (int r = 0; r < k; ++r) {
      Cand c{-INFINITY, INT_MAX};
#pragma unroll
      for (int u = 0; u < kU; ++u) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int v = vbase + u * (kTkThreads * 4) + e;
          const float val = vals[4 * u + e];
          const bool after = val < last.v || (val == last.v && v > last.i);
          if (after && val > c.v) c = Cand{val, v};
        }
      }
      const unsigned key = ordered_key(c.v);
      const unsigned kmax = __reduce_max_sync(0xffffffffu, key);
      const unsigned imin = __reduce_min_sync(0xffffffffu, key == kmax ? static_cast<unsigned>(c.i) : 0xffffffffu);
      // an exhausted warp reduces to (-inf, INT_MAX): INT_MAX is the smallest index any lane reports then
      const Cand w{key_value(kmax), static_cast<int>(imin)};
      last = w;
      if (lane == r) kept = w;
    }
    if (kept.i == INT_MAX) kept.i = kSentinel0 + (part * kWarps + warp) * kMaxK + lane;  // unique per entry
    if (lane < k) s_wl[warp * kMaxK + lane] = kept;
  }
  // ---- the warps' sorted lists are merged by counting
  __shared__ Cand s_top[kMaxK];
  __syncthreads();
  // Two threads per entry (entry = list * kMaxK + place), each searching half of the lists: with a
  // single warp per scheduler a chain of dependent instructions issues once every few cycles, so
  // the work is spread over all warps of the block.
  static_assert(kWarps == 8 && kTkSplit == 8 && kTkThreads == 2 * 8 * kMaxK, "merge layout");
  __shared__ int s_part[2][8 * kMaxK];
  const int entry = threadIdx.x & (8 * kMaxK - 1), half = threadIdx.x >> 7;
  const bool live = (entry % kMaxK) < k;
  {
    const Cand me = s_wl[entry];
    s_part[half][entry] = live ? rank_among<4>(s_wl + half * 4 * kMaxK, k, me) : 0;
    __syncthreads();
    const int rank = s_part[0][entry] + s_part[1][entry];
    if (half == 0 && live && rank < k) s_top[rank] = me;
  }
  __syncthreads();
  if (static_cast<int>(threadIdx.x) < k) kept = s_top[threadIdx.x];

  // ---- lists and (max, sum) pairs meet in the first block
  cluster.barrier_wait();
  if (static_cast<int>(threadIdx.x) < k) cluster.map_shared_rank(s_all, 0)[part * kMaxK + threadIdx.x] = kept;
  if (threadIdx.x == 0) {
    float gm = -INFINITY, gz = 0.f;
    for (int q = 0; q < kWarps; ++q) {
      const float nm = fmaxf(gm, s_m[q]);
      gz = (gm == -INFINITY ? 0.f : gz * __expf(gm - nm)) + (s_m[q] == -INFINITY ? 0.f : s_z[q] * __expf(s_m[q] - nm));
      gm = nm;
    }
    cluster.map_shared_rank(s_pm, 0)[part] = gm;
    cluster.map_shared_rank(s_pz, 0)[part] = gz;
  }
  cluster.sync();
  if (part != 0) return;
  __shared__ float s_lse;
  if (threadIdx.x == 0) {
    float gm = -INFINITY, gz = 0.f;
    for (int q = 0; q < kTkSplit; ++q) {
      const float nm = fmaxf(gm, s_pm[q]);
      gz = (gm == -INFINITY ? 0.f : gz * __expf(gm - nm)) + (s_pm[q] == -INFINITY ? 0.f : s_pz[q] * __expf(s_pm[q] - nm));
      gm = nm;
    }
    s_lse = gm + logf(gz);
  }
  __syncthreads();
  {
    const Cand me = s_all[entry];
    s_part[half][entry] = live ? rank_among<4>(s_all + half * 4 * kMaxK, k, me) : 0;
    __syncthreads();
    const int rank = s_part[0][entry] + s_part[1][entry];
    if (half == 0 && live && rank < k) {
      tokens[static_cast<int64_t>(row) * k + rank] = (me.i >= kSentinel0) ? 0 : me.i;
      logprob[static_cast<int64_t>(row) * k + rank] = me.v - s_lse;
    }
  }
}

constexpr int kRerankThreads = 1024;  // also the candidate limit

// One block per sequence, one thread per candidate. A candidate is kept iff it is the root or
// among the T - 1 best others in (score descending, index ascending) order, decided by a radix
// select on unique keys; its new label is the number of kept candidates before it in (depth,
// score descending, index ascending) order, counted with warp ballots over the kept list.
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
  __shared__ short s_par[kRerankThreads], s_label[kRerankThreads];
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
  // ---- which candidates stay: the root and the T - 1 best of the others in (score descending,
  // index ascending) order. Every candidate gets a unique 48-bit key (order-preserving score
  // bits, then 65535 - index); a radix select over six 8-bit digits finds the key of the
  // (T - 1)-th largest, and a candidate stays iff its key is not below it.
  __shared__ int s_hist[256], s_wsum[8], s_digit, s_remaining;
  unsigned long long key = 0ull;
  if (i < C && !bad) {
    int n = i;
    while (n > 0) { n = s_par[n]; ++depth; }
    if (i > 0) key = (static_cast<unsigned long long>(ordered_key(s_score[i])) << 16) | static_cast<unsigned>(65535 - i);
  }
  bool active = i > 0 && i < C && !bad;
  int remaining = T - 1;  // the wanted key is the remaining-th largest among the active ones
  unsigned long long threshold = 0ull;
  if (T > 1) {
#pragma unroll 1
    for (int shift = 40; shift >= 0; shift -= 8) {
      if (i < 256) s_hist[i] = 0;
      __syncthreads();
      const int digit = static_cast<int>((key >> shift) & 0xffull);
      if (active) atomicAdd(&s_hist[digit], 1);
      __syncthreads();
      // suffix sums over the 256 bins: above[d] = number of active keys with a larger digit
      int h = 0, incl = 0;
      if (i < 256) {
        h = s_hist[255 - i];  // thread i looks at digit 255 - i, so a forward scan is a suffix sum
        incl = h;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const int o = __shfl_up_sync(0xffffffffu, incl, off);
          if ((i & 31) >= off) incl += o;
        }
        if ((i & 31) == 31) s_wsum[i >> 5] = incl;
      }
      __syncthreads();
      if (i < 256) {
        for (int w = 0; w < (i >> 5); ++w) incl += s_wsum[w];
        const int above = incl - h;
        if (above < remaining && incl >= remaining) {  // exactly one digit satisfies this
          s_digit = 255 - i;
          s_remaining = remaining - above;
        }
      }
      __syncthreads();
      const int d = s_digit;
      remaining = s_remaining;
      threshold |= static_cast<unsigned long long>(d) << shift;
      active = active && digit == d;
    }
  }
  if (i < C && !bad) {
    keep = i == 0 || (T > 1 && key >= threshold);
    s_label[i] = keep ? 0 : -1;
  }
  __syncthreads();
  // ---- compact list of the kept candidates (any order), then labels by counting among them:
  // warp w ranks list slots 2 w and 2 w + 1, one ballot per 32 list entries
  __shared__ int s_nkept;
  __shared__ short s_kept[SPECVLM_MAX_TREE], s_kdepth[SPECVLM_MAX_TREE], s_klabel[SPECVLM_MAX_TREE];
  __shared__ float s_kscore[SPECVLM_MAX_TREE];
  if (i == 0) s_nkept = 0;
  __syncthreads();
  int my_slot = -1;
  if (keep) {
    my_slot = atomicAdd(&s_nkept, 1);
    if (my_slot < SPECVLM_MAX_TREE) {
      s_kept[my_slot] = static_cast<short>(i);
      s_kdepth[my_slot] = static_cast<short>(depth);
      s_kscore[my_slot] = s_score[i];
    }
  }
  __syncthreads();
  {
    const int nk = min(s_nkept, SPECVLM_MAX_TREE);
    const int lane = i & 31, warp = i >> 5;
#pragma unroll
    for (int sub = 0; sub < 2; ++sub) {
      const int m = 2 * warp + sub;  // warp-uniform
      if (m < nk) {
        const int mi = s_kept[m], md = s_kdepth[m];
        const float ms = s_kscore[m];
        int cnt = 0;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const int q = lane + 32 * half;
          bool first = false;
          if (q < nk && q != m) {
            const int qi = s_kept[q], qd = s_kdepth[q];
            const float qs = s_kscore[q];
            first = (qd < md) || (qd == md && (qs > ms || (qs == ms && qi < mi)));
          }
          cnt += __popc(__ballot_sync(0xffffffffu, first));
        }
        if (lane == 0) s_klabel[m] = static_cast<short>(cnt);
      }
    }
  }
  __syncthreads();
  int label = -1;
  if (keep && my_slot < SPECVLM_MAX_TREE) label = s_klabel[my_slot];
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
  const int n4 = (V + 3) / 4;
  const int per = (n4 + kTkSplit - 1) / kTkSplit;  // 16-byte groups per block of the cluster
  if (per <= 32 * kTkThreads) {
    const int vec = (V % 4 == 0) && (row_stride % 4 == 0) && aligned16(logits);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(kTkSplit) * rows);
    cfg.blockDim = dim3(kTkThreads);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kTkSplit;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e;
    if (per <= 4 * kTkThreads)  // rows of up to 32768 logits
      e = cudaLaunchKernelEx(&cfg, topk_cluster_kernel<4>, logits, V, row_stride, k, vec, tokens, logprob);
    else if (per <= 8 * kTkThreads)
      e = cudaLaunchKernelEx(&cfg, topk_cluster_kernel<8>, logits, V, row_stride, k, vec, tokens, logprob);
    else if (per <= 16 * kTkThreads)
      e = cudaLaunchKernelEx(&cfg, topk_cluster_kernel<16>, logits, V, row_stride, k, vec, tokens, logprob);
    else  // up to 262144
      e = cudaLaunchKernelEx(&cfg, topk_cluster_kernel<32>, logits, V, row_stride, k, vec, tokens, logprob);
    return check_cuda(e, "topk_logprob launch");
  }
  // longer rows: one block per row, re-reading global memory in every round
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
