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
// Two launches. (1) Row statistics: for every node row, max and sum of exp((l - max) / temperature)
// over the vocabulary in one pass over HBM; one cluster of four thread blocks per row, every
// thread keeps a running (max, sum) pair over the float4 groups it streams, pairs are merged
// through shuffles, shared memory and distributed shared memory in a fixed order. (2) The walk:
// one block of 1024 threads per sequence. Per node and in parallel: the child bit mask of its
// parent, whether an earlier sibling carries the same token, and p(token) in the parent's row
// from the row statistics. Thread 0 then walks real children only, on shared-memory values
// (one division per child). Where the walk stops an inverse-CDF search draws the token: the row
// is cut into 1024 chunks of consecutive tokens; every warp sums 32 chunks with all its loads
// in flight at once (removed tokens get weight 0), running totals come from warp scans, warp 0
// picks span, chunk and token with ballots.
#include "common.cuh"

#include <cooperative_groups.h>
#include <math.h>

namespace specvlm {

constexpr int kSampleThreads = 1024;
constexpr int kMaxChildren = SPECVLM_MAX_TREE;

constexpr int kStatThreads = 256;
constexpr int kStatSplit = 4;  // CTAs per row = cluster size

// (max, sum of exp((x - max) * inv_temp)) of a set of logits; the empty set is (-inf, 0).
struct Stat {
  float m, z;
};

__device__ __forceinline__ Stat merge(Stat a, Stat b, float inv_temp) {
  const float m = fmaxf(a.m, b.m);
  if (m == -INFINITY) return Stat{m, 0.f};
  return Stat{m, a.z * __expf((a.m - m) * inv_temp) + b.z * __expf((b.m - m) * inv_temp)};
}

// Folds up to n values (n <= 32, -inf padding allowed) into the running pair.
template <int N>
__device__ __forceinline__ void absorb(Stat& st, const float (&x)[N], float inv_temp) {
  float mloc = -INFINITY;
#pragma unroll
  for (int i = 0; i < N; ++i) mloc = fmaxf(mloc, x[i]);
  if (mloc > st.m) {  // st.m = -inf, z = 0 at the start: 0 * exp(-inf) = 0
    st.z *= __expf((st.m - mloc) * inv_temp);
    st.m = mloc;
  }
  if (st.m > -INFINITY) {
#pragma unroll
    for (int i = 0; i < N; ++i) st.z += __expf((x[i] - st.m) * inv_temp);
  }
}

__global__ void __launch_bounds__(kStatThreads)
softmax_stats_kernel(const float* __restrict__ logits, int V, float inv_temp, int vec, float2* __restrict__ stats) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  const int row = blockIdx.x / kStatSplit, part = blockIdx.x % kStatSplit;  // part == rank in the cluster
  const float* x = logits + static_cast<int64_t>(row) * V;
  grid_dependency_sync();
  cluster.barrier_arrive();  // matched by the wait before the first remote store
  Stat st{-INFINITY, 0.f};
  if (vec) {
    const float4* x4 = reinterpret_cast<const float4*>(x);
    const int n4 = V >> 2;
    const int per = (n4 + kStatSplit - 1) / kStatSplit;
    const int g0 = part * per, g1 = min(g0 + per, n4);
    for (int g = g0 + threadIdx.x; g < g1; g += 8 * kStatThreads) {
      float a[32];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int gu = g + u * kStatThreads;
        const float4 t = (gu < g1) ? __ldg(x4 + gu) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        a[4 * u] = t.x; a[4 * u + 1] = t.y; a[4 * u + 2] = t.z; a[4 * u + 3] = t.w;
      }
      absorb(st, a, inv_temp);
    }
  } else {
    const int per = (V + kStatSplit - 1) / kStatSplit;
    const int e0 = part * per, e1 = min(e0 + per, V);
    for (int e = e0 + threadIdx.x; e < e1; e += 8 * kStatThreads) {
      float a[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int eu = e + u * kStatThreads;
        a[u] = (eu < e1) ? __ldg(x + eu) : -INFINITY;
      }
      absorb(st, a, inv_temp);
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const Stat o{__shfl_xor_sync(0xffffffffu, st.m, off), __shfl_xor_sync(0xffffffffu, st.z, off)};
    st = merge(st, o, inv_temp);
  }
  constexpr int kWarps = kStatThreads / 32;
  __shared__ float sm[kStatSplit * kWarps], sz[kStatSplit * kWarps];
  cluster.barrier_wait();
  if ((threadIdx.x & 31) == 0) {
    float* dm = cluster.map_shared_rank(sm, 0);
    float* dz = cluster.map_shared_rank(sz, 0);
    dm[part * kWarps + (threadIdx.x >> 5)] = st.m;
    dz[part * kWarps + (threadIdx.x >> 5)] = st.z;
  }
  cluster.sync();
  if (part == 0 && threadIdx.x < 32) {
    Stat r{-INFINITY, 0.f};
    if (threadIdx.x < kStatSplit * kWarps) r = Stat{sm[threadIdx.x], sz[threadIdx.x]};
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const Stat o{__shfl_xor_sync(0xffffffffu, r.m, off), __shfl_xor_sync(0xffffffffu, r.z, off)};
      r = merge(r, o, inv_temp);
    }
    if (threadIdx.x == 0) stats[row] = make_float2(r.m, r.z);
  }
}

__global__ void __launch_bounds__(kSampleThreads)
accept_sample_kernel(const int32_t* __restrict__ draft, const int32_t* __restrict__ parent,
                     const float* __restrict__ logits, const float2* __restrict__ stats,
                     const float* __restrict__ u_accept, const float* __restrict__ u_sample, float inv_temp,
                     int T, int V,
                     int32_t* __restrict__ accepted_idx, int acc_stride, int32_t* __restrict__ accept_len,
                     int32_t* __restrict__ next_token, int32_t* __restrict__ status) {
  const int b = blockIdx.x;
  draft += b * T; parent += b * T; u_accept += b * T; u_sample += b * T;
  logits += static_cast<int64_t>(b) * T * V;
  stats += b * T;
  __shared__ float s_px[SPECVLM_MAX_TREE];  // p(token of node c) in its parent's row; 0 if unusable
  __shared__ float s_ua[SPECVLM_MAX_TREE], s_us[SPECVLM_MAX_TREE];
  __shared__ unsigned long long s_children[SPECVLM_MAX_TREE];  // bit c: node c is a child of this node
  __shared__ int s_draft[SPECVLM_MAX_TREE], s_usable[SPECVLM_MAX_TREE], s_path[SPECVLM_MAX_TREE];
  __shared__ int s_gone[kMaxChildren];
  __shared__ float s_chunk[kSampleThreads], s_cum[kSampleThreads], s_span[32];
  __shared__ int s_next, s_ngone, s_bad, s_result;
  const int t = threadIdx.x;
  if (t == 0) { s_bad = 0; s_ngone = 0; s_path[0] = 0; }
  if (t < SPECVLM_MAX_TREE) s_children[t] = 0ull;
  __syncthreads();
  // ---- everything the walk needs is computed per node in parallel
  int pr = -1, x = -1;
  bool bad = false;
  if (t < T) {
    pr = parent[t];
    x = draft[t];
    s_draft[t] = x;
    s_ua[t] = u_accept[t];
    s_us[t] = u_sample[t];
    bad = (t == 0) ? (pr != -1) : (pr < 0 || pr >= t);
    if (bad) s_bad = 1;
    else if (t > 0) atomicOr(&s_children[pr], 1ull << t);
  }
  __syncthreads();
  const bool bad_tree = s_bad != 0;
  if (t < T) {
    // a token is unusable if it is out of range or an earlier sibling carries it (already removed by then)
    bool usable = !bad_tree && t > 0 && x >= 0 && x < V;
    if (usable) {
      unsigned long long earlier = s_children[pr] & ((1ull << t) - 1ull);
      while (earlier != 0ull) {
        const int c = __ffsll(static_cast<long long>(earlier)) - 1;
        earlier &= earlier - 1ull;
        if (s_draft[c] == x) usable = false;
      }
    }
    s_usable[t] = usable ? 1 : 0;
  }
  // Everything above reads only this call's inputs, which no kernel that may still be running
  // writes; the row statistics come from the launch just before this one.
  const float child_logit = (t < T && s_usable[t]) ? logits[static_cast<int64_t>(pr) * V + x] : 0.f;
  grid_dependency_sync();
  if (t < T) {
    float px = 0.f;
    if (s_usable[t]) {
      const float2 mz = stats[pr];
      px = __expf((child_logit - mz.x) * inv_temp) / mz.y;
    }
    s_px[t] = px;
  }
  __syncthreads();

  // ---- the walk: sequential over real children only, on values in shared memory
  int cur = 0, depth = 0;
  if (t == 0) {
    for (int guard = 0; guard < SPECVLM_MAX_TREE; ++guard) {
      unsigned long long todo = bad_tree ? 0ull : s_children[cur];
      float removed = 0.f;
      int kept = -1;
      while (todo != 0ull) {
        const int c = __ffsll(static_cast<long long>(todo)) - 1;  // children in index order
        todo &= todo - 1ull;
        const float px = s_px[c];
        const float rest = 1.f - removed;
        if (rest > 0.f && s_ua[c] < px / rest) { kept = c; break; }
        removed += px;
      }
      if (kept < 0) break;
      cur = kept;
      s_path[++depth] = kept;
    }
    s_next = cur;
    s_result = depth;
  }
  __syncthreads();
  cur = s_next;
  depth = s_result;
  // every child of the node where the walk stopped was rejected: their tokens are removed from p
  if (t < T && t > 0 && !bad_tree && pr == cur && s_usable[t]) s_gone[atomicAdd(&s_ngone, 1)] = x;
  __syncthreads();  // also: s_result is reused for the drawn token below
  {
    const float* row = logits + static_cast<int64_t>(cur) * V;
    const float m = stats[cur].x;
    // ---- draw the next token from what is left of p: first v with cumulative weight > target.
    // The row is cut into 1024 chunks of consecutive tokens, 32 chunks (a "span") per warp.
    // Level 1: every warp sums its chunks with removed tokens left out; lane l ends up with the
    // total of chunk 32 w + l, a warp scan gives the running totals inside the span.
    // Level 2: warp 0 scans the 32 span totals, picks the span, then the chunk inside it, then
    // searches the chunk one token per lane. No step walks a list sequentially.
    const int ngone = s_ngone;
    auto is_gone = [&](int v) {
      bool gone = false;
      for (int j = 0; j < ngone; ++j) gone = gone || (s_gone[j] == v);
      return gone;
    };
    const int chunk = (V + kSampleThreads - 1) / kSampleThreads;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float xv[32];
    if (chunk <= 32) {
      // one token per lane and chunk: all 32 loads of a lane are independent and issued together
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        const int v = (warp * 32 + j) * chunk + lane;
        xv[j] = (lane < chunk && v < V) ? __ldg(row + v) : -INFINITY;
      }
      for (int q = 0; q < ngone; ++q) {  // removed tokens inside this warp's span get weight 0
        const int g = s_gone[q];
        const int c = g / chunk;
        if ((c >> 5) == warp) {
          const int jj = c & 31, ll = g - c * chunk;
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (j == jj && lane == ll) xv[j] = -INFINITY;
        }
      }
#pragma unroll
      for (int j = 0; j < 32; ++j) xv[j] = __expf((xv[j] - m) * inv_temp);
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j) xv[j] = 0.f;
      for (int off = lane; off < chunk; off += 32) {
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const int v = (warp * 32 + j) * chunk + off;
          if (v < V && !is_gone(v)) xv[j] += __expf((__ldg(row + v) - m) * inv_temp);
        }
      }
    }
    // transposing reduction: after five exchange steps lane l holds the total of chunk 32 warp + l
#pragma unroll
    for (int step = 16, n = 16; step >= 1; step >>= 1, n >>= 1) {
      const bool upper = (lane & step) != 0;
#pragma unroll
      for (int i = 0; i < n; ++i) {
        const float send = upper ? xv[i] : xv[i + n];
        const float keep = upper ? xv[i + n] : xv[i];
        xv[i] = keep + __shfl_xor_sync(0xffffffffu, send, step);
      }
    }
    const float cs = xv[0];
    float cum = cs;  // running total inside the span, this chunk included
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const float o = __shfl_up_sync(0xffffffffu, cum, off);
      if (lane >= off) cum += o;
    }
    s_chunk[threadIdx.x] = cs;
    s_cum[threadIdx.x] = cum;
    if (lane == 31) s_span[warp] = cum;
    __syncthreads();
    if (warp == 0) {
      const float sp = s_span[lane];
      float si = sp;  // running total over spans, this span included
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const float o = __shfl_up_sync(0xffffffffu, si, off);
        if (lane >= off) si += o;
      }
      const float total = __shfl_sync(0xffffffffu, si, 31);
      const float target = s_us[cur] * total;
      int res = -1;
      // span: the first whose running total passes the target, else (target at or beyond the total
      // by rounding) the last one with any weight
      const unsigned hit1 = __ballot_sync(0xffffffffu, target < si);
      const unsigned nz1 = __ballot_sync(0xffffffffu, sp > 0.f);
      const int wsel = hit1 != 0u ? __ffs(hit1) - 1 : (nz1 != 0u ? 31 - __clz(nz1) : -1);
      if (wsel >= 0) {
        const float before_span = __shfl_sync(0xffffffffu, si - sp, wsel);
        // chunk inside the span, same rule; before_span + (running total of lane 31) is the very
        // sum compared above, so a span chosen by a hit always contains a chunk that hits
        const float ccum = s_cum[wsel * 32 + lane], ccs = s_chunk[wsel * 32 + lane];
        const unsigned hit2 = __ballot_sync(0xffffffffu, target < before_span + ccum);
        const unsigned nz2 = __ballot_sync(0xffffffffu, ccs > 0.f);
        const int csel = hit2 != 0u ? __ffs(hit2) - 1 : (nz2 != 0u ? 31 - __clz(nz2) : -1);
        if (csel >= 0) {
          const float prev = __shfl_sync(0xffffffffu, ccum, csel > 0 ? csel - 1 : 0);
          float acc = csel > 0 ? before_span + prev : before_span;
          const int c = wsel * 32 + csel;
          const int a0 = c * chunk, a1 = min(a0 + chunk, V);
          for (int base = a0; base < a1; base += 32) {
            const int v = base + lane;
            const bool present = v < a1 && !is_gone(v);
            const float w = present ? __expf((row[v] - m) * inv_temp) : 0.f;
            float wi = w;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
              const float o = __shfl_up_sync(0xffffffffu, wi, off);
              if (lane >= off) wi += o;
            }
            const unsigned hits = __ballot_sync(0xffffffffu, present && (acc + wi > target));
            const unsigned pres = __ballot_sync(0xffffffffu, present);
            if (hits != 0u) { res = base + __ffs(hits) - 1; break; }
            if (pres != 0u) res = base + 31 - __clz(pres);  // last candidate that is still present
            acc += __shfl_sync(0xffffffffu, wi, 31);
          }
        }
      }
      if (res < 0 && lane == 0) {  // no weight anywhere: the last token that is still present
        for (int v = V - 1; v >= 0 && res < 0; --v)
          if (!is_gone(v)) res = v;
      }
      if (lane == 0) s_result = res;
    }
    __syncthreads();
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
                                     int32_t* next_token, float* row_stats, int32_t* status, void* stream) {
  SPECVLM_REQUIRE(B >= 0 && T >= 1 && T <= SPECVLM_MAX_TREE, "accept_sample: need B >= 0 and 1 <= T <= 64");
  SPECVLM_REQUIRE(V >= 1, "accept_sample: V must be positive");
  SPECVLM_REQUIRE(temperature > 0.f && isfinite(temperature), "accept_sample: temperature must be positive (use specvlm_accept for 0)");
  if (B == 0) return SPECVLM_OK;
  SPECVLM_REQUIRE(draft_tokens && tree_parent && target_logits && uniforms_accept && uniforms_sample &&
                      accepted_idx && accept_len && next_token && row_stats,
                  "accept_sample: null pointer");
  SPECVLM_REQUIRE((reinterpret_cast<uintptr_t>(row_stats) & 7) == 0, "accept_sample: row_stats must be 8-byte aligned");
  SPECVLM_REQUIRE(acc_stride >= 1, "accept_sample: acc_stride must be >= 1");
  const float inv_temp = 1.0f / temperature;
  float2* stats = reinterpret_cast<float2*>(row_stats);
  {
    const int vec = (V % 4 == 0) && aligned16(target_logits);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(kStatSplit) * B * T);  // rows along x: no 65535 limit
    cfg.blockDim = dim3(kStatThreads);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kStatSplit;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // the kernel starts with grid_dependency_sync()
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    const int rc = check_cuda(cudaLaunchKernelEx(&cfg, softmax_stats_kernel, target_logits, V, inv_temp, vec, stats),
                              "accept_sample row statistics launch");
    if (rc != SPECVLM_OK) return rc;
  }
  // The walk kernel is scheduled while the statistics kernel runs: it reads its own inputs, then
  // waits for the statistics.
  return check_cuda(launch_overlapped(accept_sample_kernel, dim3(B), dim3(kSampleThreads),
                                      static_cast<cudaStream_t>(stream), draft_tokens, tree_parent, target_logits,
                                      static_cast<const float2*>(stats), uniforms_accept, uniforms_sample, inv_temp,
                                      T, V, accepted_idx, acc_stride, accept_len, next_token, status),
                    "accept_sample launch");
}
