// Tree-verification attention, split-KV flash-decoding form (one layer per launch).
//
// The target verifies the whole draft tree in one pass with tree attention (Sections 3.1,
// 4.1); the cost is streaming the KV cache from HBM (Section 3.2). Each thread block takes
// one (sequence, head, KV split): it stages 64-key K/V tiles in shared memory with
// 16-byte cp.async copies (XOR-swizzled rows), computes S = Q K^T and O += P V for the
// <= 64 tree queries on the tensor cores (bf16 in, fp32 accumulate), keeps an online
// softmax per query row in registers (quad shuffles for row max / sum), and applies the
// tree mask as one 64-bit word per query row on the tiles that reach the tree slots.
// Splits of one (sequence, head) meet through fp32 partials in the workspace; the split
// that arrives last (atomic counter, no waiting) combines them and writes bf16.
#include "common.cuh"
#include "attn_params.cuh"

#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <math.h>

#include <mutex>

namespace specvlm {

constexpr int kD = SPECVLM_HEAD_DIM;  // 128
constexpr int kRows = 64;             // padded tree queries
constexpr int kTileN = 64;            // keys per tile
constexpr int kThreads = 128;         // 4 warps x 16 query rows
constexpr int kStages = 3;
constexpr int kTileBytes = kTileN * kD * 2;  // 16 KB
constexpr int kSmemBytes = kRows * kD * 2 + kStages * 2 * kTileBytes;  // 16 KB + 96 KB

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// 16-byte async copy; src_bytes = 0 zero-fills the destination without reading.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

// Byte offset of 16-byte chunk `c` of row `r` in a [rows][128] bf16 tile (256-byte rows).
__device__ __forceinline__ uint32_t swz(int r, int c) { return r * 256 + ((c ^ (r & 7)) << 4); }

// Stage keys [key0, key0 + 64) of K and V; rows at or beyond n_keys are zero-filled and
// never read from memory (their cache slots may hold arbitrary bit patterns).
__device__ __forceinline__ void load_tile(uint32_t sk, uint32_t sv, const uint16_t* kbase, const uint16_t* vbase,
                                          int64_t k_ss, int64_t v_ss, int key0, int n_keys) {
#pragma unroll
  for (int it = 0; it < (kTileN * 16) / kThreads; ++it) {
    const int idx = it * kThreads + threadIdx.x;
    const int r = idx >> 4, c = idx & 15;
    const int key = key0 + r;
    const bool in = key < n_keys;
    const int64_t row = in ? key : 0;
    cp_async16(sk + swz(r, c), kbase + row * k_ss + c * 8, in ? 16 : 0);
    cp_async16(sv + swz(r, c), vbase + row * v_ss + c * 8, in ? 16 : 0);
  }
}

// kClusterCombine = false: splits meet through the global workspace (any split count).
// kClusterCombine = true : the splits of one (sequence, head) form a thread-block cluster
// (cluster size == split count <= 8) and meet through distributed shared memory.
template <bool kClusterCombine>
__device__ __forceinline__ void tree_attn_body(const AttnParams& p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const uint32_t sq = smem_u32(smem);
  const uint32_t stage0 = sq + kRows * kD * 2;

  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t4 = lane & 3;
  const int T = p.T;

  int P = p.prefix_len[b];
  int n_keys = P + T;
  if (P < 0 || n_keys > p.S_cap) {  // skip the sequence: it contributes no keys, output is zero
    if (threadIdx.x == 0 && split == 0 && h == 0 && p.status != nullptr)
      atomicOr(p.status, SPECVLM_STATUS_BAD_PREFIX);
    P = 0;
    n_keys = 0;
  }
  const int tiles_total = (n_keys + kTileN - 1) / kTileN;
  const int tps = (tiles_total + p.splits - 1) / p.splits;
  const int tile_begin = min(split * tps, tiles_total);
  const int tile_end = min(tile_begin + tps, tiles_total);
  const int n_tiles = tile_end - tile_begin;

  const uint16_t* qbase = p.q + b * p.q_sb + h * p.q_sh;
  const uint16_t* kbase = p.k + b * p.k_sb + h * p.k_sh;
  const uint16_t* vbase = p.v + b * p.v_sb + h * p.v_sh;

  // ---- prologue: Q (rows >= T zero-filled) and the first stages
  if (n_tiles > 0) {
#pragma unroll
    for (int it = 0; it < (kRows * 16) / kThreads; ++it) {
      const int idx = it * kThreads + threadIdx.x;
      const int r = idx >> 4, c = idx & 15;
      const bool in = r < T;
      cp_async16(sq + swz(r, c), qbase + (in ? r : 0) * p.q_st + c * 8, in ? 16 : 0);
    }
  }
#pragma unroll
  for (int s = 0; s < kStages - 1; ++s) {
    if (s < n_tiles)
      load_tile(stage0 + s * 2 * kTileBytes, stage0 + s * 2 * kTileBytes + kTileBytes, kbase, vbase, p.k_ss,
                p.v_ss, (tile_begin + s) * kTileN, n_keys);
    cp_async_commit();
  }

  // ---- tree mask words of this thread's two query rows
  const int row0 = warp * 16 + g, row1 = row0 + 8;
  uint64_t mask0 = 0, mask1 = 0;
  if (p.mask != nullptr) {
    if (row0 < T) mask0 = p.mask[b * T + row0];
    if (row1 < T) mask1 = p.mask[b * T + row1];
  } else {
    const int32_t* par = p.parent + b * T;
    for (int pass = 0; pass < 2; ++pass) {
      const int row = pass ? row1 : row0;
      uint64_t bits = 0;
      if (row < T) {
        int n = row;
        for (int step = 0; step < kRows && n >= 0 && n < T; ++step) {  // bounded even for bad trees
          bits |= 1ull << n;
          const int up = par[n];
          n = (up < n) ? up : -1;
        }
      }
      if (pass) mask1 = bits; else mask0 = bits;
    }
  }
  const bool warp_active = warp * 16 < T;

  float o[16][4];
#pragma unroll
  for (int i = 0; i < 16; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  uint32_t qf[8][4];

  for (int it = 0; it < n_tiles; ++it) {
    cp_async_wait<kStages - 2>();
    __syncthreads();
    // prefetch tile it + kStages - 1 into the stage freed by tile it - 1
    {
      const int nxt = it + kStages - 1;
      if (nxt < n_tiles) {
        const uint32_t st = stage0 + (nxt % kStages) * 2 * kTileBytes;
        load_tile(st, st + kTileBytes, kbase, vbase, p.k_ss, p.v_ss, (tile_begin + nxt) * kTileN, n_keys);
      }
      cp_async_commit();
    }
    if (it == 0) {
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const int r = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        ldsm_x4(sq + swz(r, ks * 2 + (lane >> 4)), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
      }
    }
    if (!warp_active) continue;

    const uint32_t sk = stage0 + (it % kStages) * 2 * kTileBytes;
    const uint32_t sv = sk + kTileBytes;
    const int key0 = (tile_begin + it) * kTileN;

    // ---- S = Q K^T  (16 x 64 per warp)
    float s[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
      for (int jp = 0; jp < 4; ++jp) {
        uint32_t b0, b1, b2, b3;
        const int r = jp * 16 + (lane & 7) + (lane >> 4) * 8;
        ldsm_x4(sk + swz(r, ks * 2 + ((lane >> 3) & 1)), b0, b1, b2, b3);
        mma_bf16(s[2 * jp], qf[ks], b0, b1);
        mma_bf16(s[2 * jp + 1], qf[ks], b2, b3);
      }
    }

    // ---- scale (log2 domain) and mask
    const bool need_mask = key0 + kTileN > P;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float x = s[j][e] * p.scale_log2;
        if (need_mask) {
          const int key = key0 + j * 8 + t4 * 2 + (e & 1);
          const uint64_t mw = (e & 2) ? mask1 : mask0;
          const int t = key - P;
          const bool ok = (t < 0) || (t < T && ((mw >> (t & 63)) & 1ull));
          x = ok ? x : -INFINITY;
        }
        s[j][e] = x;
      }
    }

    // ---- online softmax
    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      mx0 = fmaxf(mx0, fmaxf(s[j][0], s[j][1]));
      mx1 = fmaxf(mx1, fmaxf(s[j][2], s[j][3]));
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
    const float ms0 = (mn0 == -INFINITY) ? 0.f : mn0;  // row with nothing visible so far
    const float ms1 = (mn1 == -INFINITY) ? 0.f : mn1;
    const float a0 = exp2f(m0 - ms0), a1 = exp2f(m1 - ms1);
    m0 = mn0;
    m1 = mn1;
    float sum0 = 0.f, sum1 = 0.f;
    uint32_t pf[4][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float p0 = exp2f(s[j][0] - ms0), p1 = exp2f(s[j][1] - ms0);
      const float p2 = exp2f(s[j][2] - ms1), p3 = exp2f(s[j][3] - ms1);
      sum0 += p0 + p1;
      sum1 += p2 + p3;
      pf[j >> 1][(j & 1) * 2 + 0] = pack_bf16(p0, p1);
      pf[j >> 1][(j & 1) * 2 + 1] = pack_bf16(p2, p3);
    }
    l0 = l0 * a0 + sum0;
    l1 = l1 * a1 + sum1;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      o[i][0] *= a0; o[i][1] *= a0; o[i][2] *= a1; o[i][3] *= a1;
    }

    // ---- O += P V  (16 x 128 per warp)
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
      for (int dp = 0; dp < 8; ++dp) {
        uint32_t b0, b1, b2, b3;
        const int r = ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        ldsm_x4_t(sv + swz(r, dp * 2 + (lane >> 4)), b0, b1, b2, b3);
        mma_bf16(o[2 * dp], pf[ks], b0, b1);
        mma_bf16(o[2 * dp + 1], pf[ks], b2, b3);
      }
    }
  }
  cp_async_wait<0>();

  // row sums were kept per thread; finish them across the quad
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);

  const int bh = b * p.H + h;
  if (p.splits == 1) {
    uint16_t* obase = p.out + b * p.o_sb + h * p.o_sh;
    const float i0 = l0 > 0.f ? 1.f / l0 : 0.f, i1 = l1 > 0.f ? 1.f / l1 : 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const int col = i * 8 + t4 * 2;
      if (row0 < T) *reinterpret_cast<uint32_t*>(obase + row0 * p.o_st + col) = pack_bf16(o[i][0] * i0, o[i][1] * i0);
      if (row1 < T) *reinterpret_cast<uint32_t*>(obase + row1 * p.o_st + col) = pack_bf16(o[i][2] * i1, o[i][3] * i1);
    }
    return;
  }

  if constexpr (kClusterCombine) {
    // ---- partial into this CTA's own shared memory (the K/V stages are free now)
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    __syncthreads();  // every warp is done reading the stages
    float* so = reinterpret_cast<float*>(smem + kRows * kD * 2);  // [64][128] fp32
    float* sml = so + kRows * kD;                                 // [64][2]
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      *reinterpret_cast<float2*>(so + row0 * kD + i * 8 + t4 * 2) = make_float2(o[i][0], o[i][1]);
      *reinterpret_cast<float2*>(so + row1 * kD + i * 8 + t4 * 2) = make_float2(o[i][2], o[i][3]);
    }
    if (t4 == 0) {
      *reinterpret_cast<float2*>(sml + row0 * 2) = make_float2(m0, l0);
      *reinterpret_cast<float2*>(sml + row1 * 2) = make_float2(m1, l1);
    }
    cluster.sync();  // all partials of this (sequence, head) are visible cluster-wide
    // Rows are dealt round-robin to the cluster's CTAs, then to the CTA's warps; a lane owns
    // four output columns and reads them from every CTA's shared memory.
    uint16_t* obase = p.out + b * p.o_sb + h * p.o_sh;
    const int nsplit = p.splits;  // == cluster size
    int nth = 0;
    for (int row = split; row < T; row += nsplit, ++nth) {
      if ((nth & 3) != warp) continue;
      float2 ml = make_float2(-INFINITY, 0.f);
      if (lane < nsplit) ml = *reinterpret_cast<const float2*>(cluster.map_shared_rank(sml, lane) + row * 2);
      float mstar = ml.x;
#pragma unroll
      for (int off = 4; off > 0; off >>= 1) mstar = fmaxf(mstar, __shfl_xor_sync(0xffffffffu, mstar, off));
      const float w = (ml.x == -INFINITY) ? 0.f : exp2f(ml.x - mstar);
      float lsum = w * ml.y;
#pragma unroll
      for (int off = 4; off > 0; off >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, off);
      lsum = __shfl_sync(0xffffffffu, lsum, 0);
      float4 x[8];
#pragma unroll
      for (int s = 0; s < 8; ++s)
        if (s < nsplit) x[s] = *(reinterpret_cast<const float4*>(cluster.map_shared_rank(so, s) + row * kD) + lane);
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        const float ws = __shfl_sync(0xffffffffu, w, s);
        if (s < nsplit && ws > 0.f) {
          acc.x += ws * x[s].x; acc.y += ws * x[s].y; acc.z += ws * x[s].z; acc.w += ws * x[s].w;
        }
      }
      const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
      uint2 packed;
      packed.x = pack_bf16(acc.x * inv, acc.y * inv);
      packed.y = pack_bf16(acc.z * inv, acc.w * inv);
      *reinterpret_cast<uint2*>(obase + row * p.o_st + lane * 4) = packed;
    }
    cluster.sync();  // nobody leaves while its shared memory may still be read
    return;
  }

  // ---- write this split's partial (unnormalised O, running max, running sum)
  {
    float* po = p.part_o + (static_cast<int64_t>(bh) * p.splits + split) * kRows * kD;
    float* pml = p.part_ml + (static_cast<int64_t>(bh) * p.splits + split) * kRows * 2;
    if (row0 < T) {
#pragma unroll
      for (int i = 0; i < 16; ++i)
        __stcg(reinterpret_cast<float2*>(po + row0 * kD + i * 8 + t4 * 2), make_float2(o[i][0], o[i][1]));
      if (t4 == 0) __stcg(reinterpret_cast<float2*>(pml + row0 * 2), make_float2(m0, l0));
    }
    if (row1 < T) {
#pragma unroll
      for (int i = 0; i < 16; ++i)
        __stcg(reinterpret_cast<float2*>(po + row1 * kD + i * 8 + t4 * 2), make_float2(o[i][2], o[i][3]));
      if (t4 == 0) __stcg(reinterpret_cast<float2*>(pml + row1 * 2), make_float2(m1, l1));
    }
  }
  __threadfence();
  __syncthreads();
  __shared__ int s_last;
  if (threadIdx.x == 0) {
    const int prev = atomicAdd(p.counters + bh, 1);
    s_last = (prev == p.splits - 1);
    if (s_last) p.counters[bh] = 0;  // ready for the next call; nobody else touches it now
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();

  // ---- combine: one warp per row, each lane owns 4 output columns
  {
    const float* po = p.part_o + static_cast<int64_t>(bh) * p.splits * kRows * kD;
    const float* pml = p.part_ml + static_cast<int64_t>(bh) * p.splits * kRows * 2;
    uint16_t* obase = p.out + b * p.o_sb + h * p.o_sh;
    for (int row = warp; row < T; row += kThreads / 32) {
      float mstar = -INFINITY;
      for (int s = 0; s < p.splits; ++s) mstar = fmaxf(mstar, __ldcg(pml + (s * kRows + row) * 2));
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      float lsum = 0.f;
      if (mstar != -INFINITY) {
        for (int s = 0; s < p.splits; ++s) {
          const float2 ml = __ldcg(reinterpret_cast<const float2*>(pml + (s * kRows + row) * 2));
          if (ml.x == -INFINITY) continue;
          const float w = exp2f(ml.x - mstar);
          const float4 x = __ldcg(reinterpret_cast<const float4*>(po + (static_cast<int64_t>(s) * kRows + row) * kD) + lane);
          acc.x += w * x.x; acc.y += w * x.y; acc.z += w * x.z; acc.w += w * x.w;
          lsum += w * ml.y;
        }
      }
      const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
      uint2 packed;
      packed.x = pack_bf16(acc.x * inv, acc.y * inv);
      packed.y = pack_bf16(acc.z * inv, acc.w * inv);
      *reinterpret_cast<uint2*>(obase + row * p.o_st + lane * 4) = packed;
    }
  }
}

__global__ void __launch_bounds__(kThreads) tree_attn_mma_kernel(const AttnParams p) {
  tree_attn_body<false>(p);
}

__global__ void __launch_bounds__(kThreads) tree_attn_mma_cluster_kernel(const AttnParams p) {
  tree_attn_body<true>(p);
}

constexpr int kMaxClusterSplits = 8;  // portable cluster size limit

// The tcgen05 path (attn_tc.cu) takes calls with up to 8 splits unless the descriptor asks for
// the legacy kernels; everything else runs on the mma.sync kernels in this file.
static bool wants_legacy(const specvlm_attn_desc& d) { return (d.flags & SPECVLM_ATTN_FLAG_LEGACY_MMA) != 0; }

int resolve_num_splits(const specvlm_attn_desc& d) {
  const bool legacy = wants_legacy(d);
  int splits = d.num_splits;
  const int64_t bh = static_cast<int64_t>(d.B) * d.H > 0 ? static_cast<int64_t>(d.B) * d.H : 1;
  if (splits <= 0) {
    if (legacy) {
      // about two CTAs per SM; up to twice the cluster limit is folded onto the cluster path
      const int64_t target = 2 * static_cast<int64_t>(sm_count());
      splits = static_cast<int>((target + bh - 1) / bh);
      if (splits > kMaxClusterSplits && splits <= 2 * kMaxClusterSplits) splits = kMaxClusterSplits;
    } else if (d.flags & (SPECVLM_ATTN_FLAG_INPUTS_STABLE | SPECVLM_ATTN_FLAG_HALF_SM)) {
      // launches overlap one another: few CTAs per launch, little or no split exchange
      splits = static_cast<int>((32 + bh - 1) / bh);
      if (splits > kMaxClusterSplits) splits = kMaxClusterSplits;
    } else {
      // one CTA per SM, the splits of a (sequence, head) in one cluster
      splits = static_cast<int>(sm_count() / bh);
      if (splits > kMaxClusterSplits) splits = kMaxClusterSplits;
    }
  }
  const int tile = (!legacy && splits <= kMaxClusterSplits) ? attn_tc_tile(d) : kTileN;
  const int max_tiles = (d.S_cap + tile - 1) / tile;
  if (splits > max_tiles) splits = max_tiles;
  if (splits > 64) splits = 64;
  if (splits < 1) splits = 1;
  return splits;
}

// Split counts up to the portable cluster size combine on chip and need no workspace.
static bool uses_cluster(int splits) { return splits >= 2 && splits <= kMaxClusterSplits; }

static int check_attn_desc(const specvlm_attn_desc* d) {
  SPECVLM_REQUIRE(d != nullptr, "attn desc is null");
  SPECVLM_REQUIRE(d->D == kD, "attn desc: D must be 128");
  SPECVLM_REQUIRE(d->T >= 1 && d->T <= SPECVLM_MAX_TREE, "attn desc: need 1 <= T <= 64");
  SPECVLM_REQUIRE(d->B >= 0 && d->B <= 65535 && d->H >= 1 && d->H <= 65535, "attn desc: bad B or H");
  SPECVLM_REQUIRE(d->S_cap >= d->T, "attn desc: S_cap must be >= T");
  SPECVLM_REQUIRE(d->num_splits >= 0, "attn desc: num_splits must be >= 0");
  SPECVLM_REQUIRE(d->softmax_scale >= 0.f && isfinite(d->softmax_scale), "attn desc: bad softmax_scale");
  const int64_t st[] = {d->q_stride_b, d->q_stride_h, d->q_stride_t, d->k_stride_b, d->k_stride_h, d->k_stride_s,
                        d->v_stride_b, d->v_stride_h, d->v_stride_s, d->o_stride_b, d->o_stride_h, d->o_stride_t};
  for (int64_t s : st) SPECVLM_REQUIRE(s >= 0 && (s % 8) == 0, "attn desc: strides must be non-negative multiples of 8");
  SPECVLM_REQUIRE(d->q_stride_t >= kD && d->k_stride_s >= kD && d->v_stride_s >= kD && d->o_stride_t >= kD,
                  "attn desc: row strides must be >= D");
  return SPECVLM_OK;
}

static size_t counters_bytes(const specvlm_attn_desc& d) {
  const size_t raw = static_cast<size_t>(d.B) * d.H * sizeof(int32_t);
  return (raw + 255) / 256 * 256;
}

}  // namespace specvlm

using namespace specvlm;

extern "C" int specvlm_attn_workspace_bytes(const specvlm_attn_desc* desc, size_t* bytes) {
  int rc = check_attn_desc(desc);
  if (rc != SPECVLM_OK) return rc;
  SPECVLM_REQUIRE(bytes != nullptr, "attn_workspace_bytes: null result pointer");
  const size_t splits = resolve_num_splits(*desc);
  const size_t bh = static_cast<size_t>(desc->B) * desc->H;
  if (splits == 1 || uses_cluster(static_cast<int>(splits)))
    *bytes = 0;
  else
    *bytes = counters_bytes(*desc) + bh * splits * kRows * 2 * sizeof(float) + bh * splits * kRows * kD * sizeof(float);
  return SPECVLM_OK;
}

extern "C" int specvlm_tree_verify_attn(const uint16_t* q, const uint16_t* k_cache, const uint16_t* v_cache,
                                        const int32_t* prefix_len, const int32_t* tree_parent,
                                        const uint64_t* tree_mask_bits, uint16_t* out,
                                        const specvlm_attn_desc* desc, void* workspace, int32_t* status,
                                        void* stream) {
  int rc = check_attn_desc(desc);
  if (rc != SPECVLM_OK) return rc;
  if (desc->B == 0) return SPECVLM_OK;
  SPECVLM_REQUIRE(q && k_cache && v_cache && prefix_len && out, "tree_verify_attn: null pointer");
  SPECVLM_REQUIRE(tree_mask_bits != nullptr || tree_parent != nullptr,
                  "tree_verify_attn: need tree_mask_bits or tree_parent");
  SPECVLM_REQUIRE(aligned16(q) && aligned16(k_cache) && aligned16(v_cache) && aligned16(out),
                  "tree_verify_attn: q/k/v/out must be 16-byte aligned");
  const int splits = resolve_num_splits(*desc);
  const bool cluster = uses_cluster(splits);
  SPECVLM_REQUIRE(splits == 1 || cluster || (workspace != nullptr && aligned16(workspace)),
                  "tree_verify_attn: workspace required (16-byte aligned) when KV is split more than 8 ways");

  AttnParams p;
  p.q = q; p.k = k_cache; p.v = v_cache; p.out = out;
  p.prefix_len = prefix_len; p.parent = tree_parent; p.mask = tree_mask_bits; p.status = status;
  p.counters = static_cast<int32_t*>(workspace);
  const size_t bh = static_cast<size_t>(desc->B) * desc->H;
  p.part_ml = workspace ? reinterpret_cast<float*>(static_cast<char*>(workspace) + counters_bytes(*desc)) : nullptr;
  p.part_o = workspace ? p.part_ml + bh * splits * kRows * 2 : nullptr;
  p.B = desc->B; p.H = desc->H; p.T = desc->T; p.S_cap = desc->S_cap; p.splits = splits;
  p.flags = desc->flags;
  const float scale = desc->softmax_scale > 0.f ? desc->softmax_scale : 1.0f / sqrtf(static_cast<float>(kD));
  p.scale_log2 = scale * 1.4426950408889634f;
  p.q_sb = desc->q_stride_b; p.q_sh = desc->q_stride_h; p.q_st = desc->q_stride_t;
  p.k_sb = desc->k_stride_b; p.k_sh = desc->k_stride_h; p.k_ss = desc->k_stride_s;
  p.v_sb = desc->v_stride_b; p.v_sh = desc->v_stride_h; p.v_ss = desc->v_stride_s;
  p.o_sb = desc->o_stride_b; p.o_sh = desc->o_stride_h; p.o_st = desc->o_stride_t;

  // Raising the dynamic shared memory limit is per function and per device.
  static bool attr_set[64] = {};
  static std::mutex attr_mu;
  std::lock_guard<std::mutex> attr_lock(attr_mu);
  int dev = 0;
  rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice");
  if (rc != SPECVLM_OK) return rc;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    rc = check_cuda(cudaFuncSetAttribute(tree_attn_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes),
                    "attn smem attribute");
    if (rc != SPECVLM_OK) return rc;
    rc = check_cuda(cudaFuncSetAttribute(tree_attn_mma_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kSmemBytes),
                    "attn smem attribute (cluster)");
    if (rc != SPECVLM_OK) return rc;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  if (!wants_legacy(*desc) && splits <= kMaxClusterSplits && attn_tc_available())
    return launch_attn_tc(p, *desc, static_cast<cudaStream_t>(stream));

  dim3 grid(splits, desc->H, desc->B);
  if (cluster) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = splits;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return check_cuda(cudaLaunchKernelEx(&cfg, tree_attn_mma_cluster_kernel, p), "tree_verify_attn cluster launch");
  }
  tree_attn_mma_kernel<<<grid, kThreads, kSmemBytes, static_cast<cudaStream_t>(stream)>>>(p);
  return check_cuda(cudaGetLastError(), "tree_verify_attn launch");
}

// ---------------------------------------------------------------------------------------------
// Variant of the split-KV attention call that needs no scratch memory from the caller.
//
// Who it is for: callers that cannot obtain device memory at the point of the call. Typical
// cases are a serving engine that handed the whole of HBM to its KV-cache block pool at
// start-up (a later cudaMalloc fails or forces the pool to shrink), a decode loop that must not
// take the device-wide synchronisation an allocation implies, and plug-in code that is given
// raw input/output pointers but no allocator. For them the split-KV partials and arrival
// counters live in the fixed device array below, which every GPU that loads this library keeps
// until the process exits.
namespace specvlm {

constexpr int kStaticMaxBH = 1024;     // sequences x heads
constexpr int kStaticMaxUnits = 512;   // sequences x heads x splits
constexpr size_t kStaticCounterBytes = kStaticMaxBH * sizeof(int32_t);
constexpr size_t kStaticMlBytes = static_cast<size_t>(kStaticMaxUnits) * kRows * 2 * sizeof(float);
constexpr size_t kStaticOBytes = static_cast<size_t>(kStaticMaxUnits) * kRows * kD * sizeof(float);
constexpr size_t kStaticBytes = kStaticCounterBytes + kStaticMlBytes + kStaticOBytes;  // ~16.3 MiB

static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

// In host code `g_static_scratch` is only a handle for the runtime, not a device address; the
// address a kernel may use comes from cudaGetSymbolAddress, asked once per device with that
// device current.
static int static_scratch_address(unsigned char** out) {
  static unsigned char* addr[64] = {};
  static std::mutex mu;
  int dev = 0;
  int rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice");
  if (rc != SPECVLM_OK) return rc;
  if (dev < 0 || dev >= 64) return fail(SPECVLM_ERR_UNSUPPORTED, "static scratch: device index out of range");
  std::lock_guard<std::mutex> lock(mu);
  if (addr[dev] == nullptr) {
    void* p = nullptr;
    rc = check_cuda(cudaGetSymbolAddress(&p, g_static_scratch), "cudaGetSymbolAddress(static scratch)");
    if (rc != SPECVLM_OK) return rc;
    if (p == nullptr) return fail(SPECVLM_ERR_CUDA, "static scratch: null symbol address");
    rc = check_cuda(cudaFuncSetAttribute(tree_attn_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kSmemBytes),
                    "attn smem attribute");
    if (rc != SPECVLM_OK) return rc;
    addr[dev] = static_cast<unsigned char*>(p);
  }
  *out = addr[dev];
  return SPECVLM_OK;
}

}  // namespace specvlm

extern "C" int specvlm_tree_verify_attn_static(const uint16_t* q, const uint16_t* k_cache,
                                               const uint16_t* v_cache, const int32_t* prefix_len,
                                               const int32_t* tree_parent, const uint64_t* tree_mask_bits,
                                               uint16_t* out, const specvlm_attn_desc* desc, int32_t* status,
                                               void* stream) {
  int rc = check_attn_desc(desc);
  if (rc != SPECVLM_OK) return rc;
  if (desc->B == 0) return SPECVLM_OK;
  SPECVLM_REQUIRE(q && k_cache && v_cache && prefix_len && out, "tree_verify_attn_static: null pointer");
  SPECVLM_REQUIRE(tree_mask_bits != nullptr || tree_parent != nullptr,
                  "tree_verify_attn_static: need tree_mask_bits or tree_parent");
  SPECVLM_REQUIRE(aligned16(q) && aligned16(k_cache) && aligned16(v_cache) && aligned16(out),
                  "tree_verify_attn_static: q/k/v/out must be 16-byte aligned");
  const int splits = resolve_num_splits(*desc);
  const int64_t bh = static_cast<int64_t>(desc->B) * desc->H;
  if (bh > kStaticMaxBH || bh * splits > kStaticMaxUnits)
    return fail(SPECVLM_ERR_UNSUPPORTED,
                "tree_verify_attn_static: B*H = " + std::to_string(bh) + " with " + std::to_string(splits) +
                    " KV splits exceeds the built-in scratch (limits: B*H <= " + std::to_string(kStaticMaxBH) +
                    ", B*H*splits <= " + std::to_string(kStaticMaxUnits) +
                    "); lower desc.num_splits or use specvlm_tree_verify_attn with a workspace");
  unsigned char* scratch = nullptr;
  rc = static_scratch_address(&scratch);
  if (rc != SPECVLM_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // The array keeps whatever the previous call left; the arrival counters must start at zero.
  rc = check_cuda(cudaMemsetAsync(scratch, 0, kStaticCounterBytes, s), "static scratch counter clear");
  if (rc != SPECVLM_OK) return rc;

  AttnParams p;
  p.q = q; p.k = k_cache; p.v = v_cache; p.out = out;
  p.prefix_len = prefix_len; p.parent = tree_parent; p.mask = tree_mask_bits; p.status = status;
  p.counters = reinterpret_cast<int32_t*>(scratch);
  p.part_ml = reinterpret_cast<float*>(scratch + kStaticCounterBytes);
  p.part_o = reinterpret_cast<float*>(scratch + kStaticCounterBytes + kStaticMlBytes);
  p.B = desc->B; p.H = desc->H; p.T = desc->T; p.S_cap = desc->S_cap; p.splits = splits;
  p.flags = desc->flags;
  const float scale = desc->softmax_scale > 0.f ? desc->softmax_scale : 1.0f / sqrtf(static_cast<float>(kD));
  p.scale_log2 = scale * 1.4426950408889634f;
  p.q_sb = desc->q_stride_b; p.q_sh = desc->q_stride_h; p.q_st = desc->q_stride_t;
  p.k_sb = desc->k_stride_b; p.k_sh = desc->k_stride_h; p.k_ss = desc->k_stride_s;
  p.v_sb = desc->v_stride_b; p.v_sh = desc->v_stride_h; p.v_ss = desc->v_stride_s;
  p.o_sb = desc->o_stride_b; p.o_sh = desc->o_stride_h; p.o_st = desc->o_stride_t;
  dim3 grid(splits, desc->H, desc->B);
  tree_attn_mma_kernel<<<grid, kThreads, kSmemBytes, s>>>(p);
  return check_cuda(cudaGetLastError(), "tree_verify_attn_static launch");
}
