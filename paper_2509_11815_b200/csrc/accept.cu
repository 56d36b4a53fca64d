// Tree metadata, lossless temperature-0 acceptance (parent-pointer path walk) and
// in-place compaction of the kept nodes' K/V rows.
//
// Acceptance rule (Section 3.1: incorrect drafted tokens are discarded; the abstract:
// lossless): node i > 0 is kept iff its drafted token equals the target's greedy token at
// its parent and the parent is kept. The result is the deepest kept node, lowest index
// among equals, and its root path.
#include "common.cuh"

namespace specvlm {

int launch_argmax(const float* logits, int rows, int V, int64_t row_stride, int32_t* out,
                  cudaStream_t stream);

constexpr int kMaxT = SPECVLM_MAX_TREE;

// ------------------------------------------------------------------ tree metadata

__global__ void tree_build_kernel(const int32_t* __restrict__ parent, const int32_t* __restrict__ prefix_len,
                                  int B, int T, uint64_t* __restrict__ mask_bits,
                                  int32_t* __restrict__ depth, int32_t* __restrict__ pos,
                                  int32_t* __restrict__ status) {
  const int b = blockIdx.x;
  const int i = threadIdx.x;
  __shared__ int s_parent[kMaxT];
  __shared__ int s_bad;
  grid_dependency_sync();
  if (i == 0) s_bad = 0;
  __syncthreads();
  if (i < T) {
    const int p = parent[b * T + i];
    s_parent[i] = p;
    if ((i == 0 && p != -1) || (i > 0 && (p < 0 || p >= i))) s_bad = 1;
  }
  __syncthreads();
  if (i >= T) return;
  uint64_t bits = 1ull << i;
  int d = 0;
  if (!s_bad) {
    int n = s_parent[i];
    while (n >= 0) {  // parent < child, so at most i steps
      bits |= 1ull << n;
      n = s_parent[n];
      ++d;
    }
  } else if (i == 0 && status != nullptr) {
    atomicOr(status, SPECVLM_STATUS_BAD_TREE);
  }
  mask_bits[b * T + i] = bits;
  if (depth != nullptr) depth[b * T + i] = d;
  if (pos != nullptr) pos[b * T + i] = (prefix_len != nullptr ? prefix_len[b] : 0) + d;
}

// ------------------------------------------------------------------ path walk

struct WalkResult {
  int depth;  // kept drafted tokens
  int node;   // deepest kept node
};

// Runs on the first 64 threads of a block (all threads of the block must call it: it
// contains block-wide barriers). s_path[0..depth] receives the kept root path.
__device__ WalkResult walk_tree(const int32_t* __restrict__ draft, const int32_t* __restrict__ parent,
                                const int32_t* __restrict__ tok, int T, int* s_parent, int* s_ok,
                                int* s_path, int* s_scratch, int32_t* status) {
  const int i = threadIdx.x;
  if (i == 0) {
    s_scratch[0] = 0;  // best key
    s_scratch[1] = 0;  // bad-tree flag
  }
  __syncthreads();
  if (i < T) {
    const int p = parent[i];
    s_parent[i] = p;
    bool bad = (i == 0) ? (p != -1) : (p < 0 || p >= i);
    if (bad) s_scratch[1] = 1;
    s_ok[i] = (i == 0) || (!bad && draft[i] == tok[p]);
  }
  __syncthreads();
  const bool bad_tree = s_scratch[1] != 0;
  if (i < T && !bad_tree) {
    bool good = true;
    int d = 0;
    int n = i;
    while (n > 0) {
      good = good && (s_ok[n] != 0);
      n = s_parent[n];
      ++d;
    }
    // deeper wins; among equal depths the lower index wins
    if (good) atomicMax(&s_scratch[0], d * kMaxT + (kMaxT - 1 - i));
  }
  __syncthreads();
  WalkResult r;
  const int key = s_scratch[0];
  r.depth = bad_tree ? 0 : key / kMaxT;
  r.node = bad_tree ? 0 : (kMaxT - 1 - key % kMaxT);
  if (i == 0) {
    if (bad_tree && status != nullptr) atomicOr(status, SPECVLM_STATUS_BAD_TREE);
    int n = r.node;
    for (int j = r.depth; j >= 0; --j) {
      s_path[j] = n;
      n = (j > 0) ? s_parent[n] : n;
    }
  }
  __syncthreads();
  return r;
}

__device__ void write_accept_outputs(const WalkResult& r, const int* s_path, const int32_t* tok, int b,
                                     int32_t* accepted_idx, int acc_stride, int32_t* accept_len,
                                     int32_t* next_token) {
  for (int j = threadIdx.x; j < acc_stride; j += blockDim.x)
    accepted_idx[static_cast<int64_t>(b) * acc_stride + j] = (j <= r.depth) ? s_path[j] : -1;
  if (threadIdx.x == 0) {
    accept_len[b] = r.depth;
    next_token[b] = tok[r.node];
  }
}

__global__ void __launch_bounds__(kMaxT)
accept_kernel(const int32_t* __restrict__ draft, const int32_t* __restrict__ parent,
              const int32_t* __restrict__ tok, int T, int32_t* __restrict__ accepted_idx, int acc_stride,
              int32_t* __restrict__ accept_len, int32_t* __restrict__ next_token,
              int32_t* __restrict__ status) {
  __shared__ int s_parent[kMaxT], s_ok[kMaxT], s_path[kMaxT], s_scratch[2];
  const int b = blockIdx.x;
  grid_dependency_sync();
  WalkResult r = walk_tree(draft + b * T, parent + b * T, tok + b * T, T, s_parent, s_ok, s_path,
                           s_scratch, status);
  write_accept_outputs(r, s_path, tok + b * T, b, accepted_idx, acc_stride, accept_len, next_token);
}

// ------------------------------------------------------------------ KV compaction

struct KvParams {
  uint16_t* k;
  uint16_t* v;
  int L, B, H, S_cap;
  int64_t stride_l, stride_b, stride_h, stride_s;
};

// Moves rows for the units [unit_begin, unit_end) of sequence b. A unit is one
// (layer, K|V, head); 16 consecutive lanes own one unit and lane c owns the c-th 16-byte
// column of every row (D = 128 bf16 = 16 columns), so a lane's copies never depend on
// another lane's. Rows go in ascending j. Path indices increase strictly, hence slot
// P + j is never a source of a later row, and sources of earlier rows were already read:
// the ascending order gives the same bytes as "read all sources, then write".
__device__ void move_rows(const KvParams& p, int b, int P, int n, const int* s_path, int first_unit,
                          int unit_stride) {
  const int lane16 = threadIdx.x & 15;
  const int units = p.L * 2 * p.H;
  for (int u = first_unit + (threadIdx.x >> 4); u < units; u += unit_stride) {
    const int h = u % p.H;
    const int kv = (u / p.H) & 1;
    const int l = u / (2 * p.H);
    uint16_t* base = (kv ? p.v : p.k) + l * p.stride_l + b * p.stride_b + h * p.stride_h;
    uint4* col = reinterpret_cast<uint4*>(base) + lane16;
    const int64_t row_u4 = p.stride_s / 8;
    for (int j0 = 1; j0 <= n; j0 += 8) {
      uint4 r[8];
#pragma unroll
      for (int q = 0; q < 8; ++q)
        if (j0 + q <= n) r[q] = col[(P + s_path[j0 + q]) * row_u4];
#pragma unroll
      for (int q = 0; q < 8; ++q)
        if (j0 + q <= n) col[(P + j0 + q) * row_u4] = r[q];
    }
  }
}

// Checks accept data that arrives from memory (standalone compaction).
__device__ bool path_ok(int P, int n, const int* s_path, int S_cap) {
  if (P < 0 || n < 0 || n >= kMaxT || P + n >= S_cap) return false;
  int prev = 0;
  for (int j = 1; j <= n; ++j) {
    const int s = s_path[j];
    if (s <= prev || s >= kMaxT || P + s >= S_cap) return false;
    prev = s;
  }
  return true;
}

constexpr int kCompactThreads = 256;

__global__ void __launch_bounds__(kCompactThreads)
kv_compact_kernel(KvParams p, const int32_t* __restrict__ prefix_len, const int32_t* __restrict__ accepted_idx,
                  int acc_stride, const int32_t* __restrict__ accept_len, int32_t* __restrict__ new_prefix_len,
                  int32_t* __restrict__ status) {
  __shared__ int s_path[kMaxT];
  __shared__ int s_good;
  const int b = blockIdx.y;
  grid_dependency_sync();
  const int P = prefix_len[b];
  const int n = accept_len[b];
  if (threadIdx.x < kMaxT)
    s_path[threadIdx.x] = (threadIdx.x < acc_stride && threadIdx.x <= n && n < kMaxT)
                              ? accepted_idx[static_cast<int64_t>(b) * acc_stride + threadIdx.x] : -1;
  __syncthreads();
  if (threadIdx.x == 0) {
    s_good = (n < acc_stride) && path_ok(P, n, s_path, p.S_cap) && s_path[0] == 0;
    if (blockIdx.x == 0) {
      if (!s_good && status != nullptr) atomicOr(status, SPECVLM_STATUS_BAD_ACCEPT);
      new_prefix_len[b] = s_good ? P + 1 + n : P;
    }
  }
  __syncthreads();
  if (!s_good) return;
  move_rows(p, b, P, n, s_path, blockIdx.x * (kCompactThreads / 16), gridDim.x * (kCompactThreads / 16));
}

__global__ void __launch_bounds__(kCompactThreads)
accept_compact_kernel(const int32_t* __restrict__ draft, const int32_t* __restrict__ parent,
                      const int32_t* __restrict__ tok, int T, KvParams p,
                      const int32_t* __restrict__ prefix_len, int32_t* __restrict__ accepted_idx, int acc_stride,
                      int32_t* __restrict__ accept_len, int32_t* __restrict__ next_token,
                      int32_t* __restrict__ new_prefix_len, int32_t* __restrict__ status) {
  __shared__ int s_parent[kMaxT], s_ok[kMaxT], s_path[kMaxT], s_scratch[2];
  const int b = blockIdx.y;
  grid_dependency_sync();
  const int P = prefix_len[b];
  WalkResult r = walk_tree(draft + b * T, parent + b * T, tok + b * T, T, s_parent, s_ok, s_path,
                           s_scratch, blockIdx.x == 0 ? status : nullptr);
  const bool prefix_ok = (P >= 0 && P + T <= p.S_cap);
  if (blockIdx.x == 0) {
    write_accept_outputs(r, s_path, tok + b * T, b, accepted_idx, acc_stride, accept_len, next_token);
    if (threadIdx.x == 0) {
      new_prefix_len[b] = prefix_ok ? P + 1 + r.depth : P;
      if (!prefix_ok && status != nullptr) atomicOr(status, SPECVLM_STATUS_BAD_PREFIX);
    }
  }
  if (!prefix_ok) return;
  move_rows(p, b, P, r.depth, s_path, blockIdx.x * (kCompactThreads / 16),
            gridDim.x * (kCompactThreads / 16));
}

static int check_kv_desc(const specvlm_kv_desc* d, const void* k, const void* v) {
  SPECVLM_REQUIRE(d != nullptr, "kv desc is null");
  SPECVLM_REQUIRE(d->D == SPECVLM_HEAD_DIM, "kv desc: D must be 128");
  SPECVLM_REQUIRE(d->L >= 1 && d->B >= 0 && d->H >= 1 && d->S_cap >= 1, "kv desc: bad shape");
  SPECVLM_REQUIRE(k != nullptr && v != nullptr, "kv caches are null");
  SPECVLM_REQUIRE(aligned16(k) && aligned16(v), "kv caches must be 16-byte aligned");
  SPECVLM_REQUIRE(d->stride_s >= d->D && (d->stride_s % 8) == 0 && (d->stride_h % 8) == 0 &&
                      (d->stride_b % 8) == 0 && (d->stride_l % 8) == 0,
                  "kv desc: strides must be multiples of 8 elements and stride_s >= D");
  return SPECVLM_OK;
}

static KvParams make_kv_params(uint16_t* k, uint16_t* v, const specvlm_kv_desc* d) {
  KvParams p;
  p.k = k; p.v = v;
  p.L = d->L; p.B = d->B; p.H = d->H; p.S_cap = d->S_cap;
  p.stride_l = d->stride_l; p.stride_b = d->stride_b; p.stride_h = d->stride_h; p.stride_s = d->stride_s;
  return p;
}

static int compact_grid_x(const specvlm_kv_desc* d) {
  const int units = d->L * 2 * d->H;
  const int per_block = kCompactThreads / 16;
  int gx = (units + per_block - 1) / per_block;
  const int cap = 4 * sm_count();
  return gx < 1 ? 1 : (gx > cap ? cap : gx);
}

}  // namespace specvlm

using namespace specvlm;

extern "C" int specvlm_tree_build(const int32_t* tree_parent, const int32_t* prefix_len, int B, int T,
                                  uint64_t* mask_bits, int32_t* depth, int32_t* pos, int32_t* status,
                                  void* stream) {
  SPECVLM_REQUIRE(B >= 0 && T >= 1 && T <= kMaxT, "tree_build: need B >= 0 and 1 <= T <= 64");
  if (B == 0) return SPECVLM_OK;
  SPECVLM_REQUIRE(tree_parent != nullptr && mask_bits != nullptr, "tree_build: null pointer");
  SPECVLM_REQUIRE(pos == nullptr || prefix_len != nullptr, "tree_build: pos needs prefix_len");
  return check_cuda(launch_overlapped(tree_build_kernel, dim3(B), dim3(kMaxT), static_cast<cudaStream_t>(stream),
                                      tree_parent, prefix_len, B, T, mask_bits, depth, pos, status),
                    "tree_build launch");
}

extern "C" int specvlm_accept(const int32_t* draft_tokens, const int32_t* tree_parent,
                              const float* target_logits, int32_t* argmax_tokens, int B, int T, int V,
                              int32_t* accepted_idx, int acc_stride, int32_t* accept_len,
                              int32_t* next_token, int32_t* status, void* stream) {
  SPECVLM_REQUIRE(B >= 0 && T >= 1 && T <= kMaxT, "accept: need B >= 0 and 1 <= T <= 64");
  if (B == 0) return SPECVLM_OK;
  SPECVLM_REQUIRE(draft_tokens && tree_parent && argmax_tokens && accepted_idx && accept_len && next_token,
                  "accept: null pointer");
  SPECVLM_REQUIRE(acc_stride >= 1, "accept: acc_stride must be >= 1");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (target_logits != nullptr) {
    SPECVLM_REQUIRE(V >= 1 && (V & 3) == 0, "accept: with logits, V must be a positive multiple of 4");
    SPECVLM_REQUIRE(aligned16(target_logits), "accept: target_logits must be 16-byte aligned");
    int rc = launch_argmax(target_logits, B * T, V, V, argmax_tokens, s);
    if (rc != SPECVLM_OK) return rc;
  }
  return check_cuda(launch_overlapped(accept_kernel, dim3(B), dim3(kMaxT), s, draft_tokens, tree_parent,
                                      static_cast<const int32_t*>(argmax_tokens), T, accepted_idx, acc_stride,
                                      accept_len, next_token, status),
                    "accept launch");
}

extern "C" int specvlm_kv_compact(uint16_t* k_cache, uint16_t* v_cache, const specvlm_kv_desc* desc,
                                  const int32_t* prefix_len, const int32_t* accepted_idx, int acc_stride,
                                  const int32_t* accept_len, int32_t* new_prefix_len, int32_t* status,
                                  void* stream) {
  int rc = check_kv_desc(desc, k_cache, v_cache);
  if (rc != SPECVLM_OK) return rc;
  if (desc->B == 0) return SPECVLM_OK;
  SPECVLM_REQUIRE(prefix_len && accepted_idx && accept_len && new_prefix_len, "kv_compact: null pointer");
  SPECVLM_REQUIRE(new_prefix_len != prefix_len, "kv_compact: new_prefix_len must not alias prefix_len");
  SPECVLM_REQUIRE(acc_stride >= 1, "kv_compact: acc_stride must be >= 1");
  dim3 grid(compact_grid_x(desc), desc->B);
  return check_cuda(launch_overlapped(kv_compact_kernel, grid, dim3(kCompactThreads), static_cast<cudaStream_t>(stream),
                                      make_kv_params(k_cache, v_cache, desc), prefix_len, accepted_idx, acc_stride,
                                      accept_len, new_prefix_len, status),
                    "kv_compact launch");
}

extern "C" int specvlm_accept_compact(const int32_t* draft_tokens, const int32_t* tree_parent,
                                      const int32_t* argmax_tokens, int T, uint16_t* k_cache,
                                      uint16_t* v_cache, const specvlm_kv_desc* desc,
                                      const int32_t* prefix_len, int32_t* accepted_idx, int acc_stride,
                                      int32_t* accept_len, int32_t* next_token, int32_t* new_prefix_len,
                                      int32_t* status, void* stream) {
  int rc = check_kv_desc(desc, k_cache, v_cache);
  if (rc != SPECVLM_OK) return rc;
  SPECVLM_REQUIRE(T >= 1 && T <= kMaxT, "accept_compact: need 1 <= T <= 64");
  if (desc->B == 0) return SPECVLM_OK;
  SPECVLM_REQUIRE(draft_tokens && tree_parent && argmax_tokens && prefix_len && accepted_idx && accept_len &&
                      next_token && new_prefix_len,
                  "accept_compact: null pointer");
  SPECVLM_REQUIRE(new_prefix_len != prefix_len, "accept_compact: new_prefix_len must not alias prefix_len");
  SPECVLM_REQUIRE(acc_stride >= 1, "accept_compact: acc_stride must be >= 1");
  dim3 grid(compact_grid_x(desc), desc->B);
  return check_cuda(launch_overlapped(accept_compact_kernel, grid, dim3(kCompactThreads),
                                      static_cast<cudaStream_t>(stream), draft_tokens, tree_parent, argmax_tokens, T,
                                      make_kv_params(k_cache, v_cache, desc), prefix_len, accepted_idx, acc_stride,
                                      accept_len, next_token, new_prefix_len, status),
                    "accept_compact launch");
}
