// Tree-verification attention on the Blackwell tensor path (sm_100a): tcgen05.mma with TMEM
// accumulators, TMA-staged K/V tiles, warp-specialised roles, cluster/DSMEM split combine.
//
// What it computes is the same as the legacy kernel: tree attention of the <= 64 draft-tree
// queries over the KV prefix plus the tree's own slots (Sections 3.1, 4.1), streaming the KV
// cache once from HBM (Section 3.2).
//
// One CTA per (sequence, head, split); the splits of one (sequence, head) are one thread-block
// cluster. Roles inside a CTA (192 threads):
//   warp 0      TMA producer: Q once, then 128-key K and V tiles into a 3-stage ring
//               (cp.async.bulk.tensor, 128-byte swizzle, no multicast); owns the TMEM allocation
//   warp 1      one lane issues tcgen05.mma: S = Q K^T (M=64, N=128, K=16 x 8) into one of two
//               TMEM buffers, O += P V (M=64, N=128, K=16 x 8); tcgen05.commit signals mbarriers
//   warps 2..5  softmax: tcgen05.ld of their 16 rows of S, scale, tree mask (one 64-bit word per
//               row, applied with selects), running max with a lazy rescale of O in TMEM, exp2,
//               bf16 P written to shared memory in the K-major swizzled operand layout
// Key tiles are anchored at the END of the sequence (tile j covers keys
// [n - 128 (j+1), n - 128 j)): the tree slots always fall in the last tile, the first tile may
// start at a negative key index, which TMA fills with zeros, and no tile ever contains a cache
// slot beyond prefix + T, so uninitialised slots are never loaded.
// Every mbarrier wait is bounded; a wait that gives up sets SPECVLM_STATUS_TIMEOUT, the CTA
// still reaches the cluster barriers, frees its TMEM and returns.
#include "attn_params.cuh"

#include <cooperative_groups.h>
#include <cuda.h>
#include <cuda_bf16.h>
#include <math.h>

#include <mutex>

namespace specvlm {

namespace tc {

constexpr int kD = SPECVLM_HEAD_DIM;
constexpr int kRows = 64;      // MMA M: padded tree queries
constexpr int kTile = 128;     // keys per tile
constexpr int kStages = 3;
constexpr int kThreads = 192;
constexpr int kSoftmaxWarp0 = 2;
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr float kRescaleThreshold = 8.0f;  // log2 units; P stays <= 2^8

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int kQBytes = kRows * kD * 2;        // 16 KB: two 64x64 swizzle atoms
constexpr int kPBytes = kRows * kTile * 2;     // 16 KB: two 64x64 swizzle atoms
constexpr int kKBytes = kTile * kD * 2;        // 32 KB: two 128x64 boxes
constexpr int kVBytes = kTile * kD * 2;        // 32 KB
constexpr int kStageBytes = kKBytes + kVBytes;
constexpr int kOffQ = 0;
constexpr int kOffP = kOffQ + kQBytes;
constexpr int kOffStage = kOffP + kPBytes;
constexpr int kOffBar = kOffStage + kStages * kStageBytes;
constexpr int kNumBars = 3 * kStages + 2 + 2 + 1 + 1 + 1;
constexpr int kOffMisc = kOffBar + kNumBars * 8;
constexpr int kSmemBytes = kOffMisc + 64 + 1024;  // + alignment slack
static_assert(kSmemBytes <= 232448, "shared memory budget");

// TMEM columns: S0 [0,128), S1 [128,256), O [256,384); 512 allocated (power of two)
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS0 = 0, kColS1 = 128, kColO = 256;

// tcgen05 instruction descriptor, kind::f16: fp32 accumulate, bf16 A and B, M=64, N=128
constexpr uint32_t make_idesc(bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | ((b_mn_major ? 1u : 0u) << 16) |
         ((128u >> 3) << 17) | ((64u >> 4) << 24);
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- mbarrier
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false after kSpinLimit unsuccessful polls or once another role has given up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 1023u) == 1023u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

// ---- TMA
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                            int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}

// ---- tcgen05
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

// Shared-memory matrix descriptor (sm_100 format, 128-byte swizzle). Offsets in bytes.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr >> 4) & 0x3FFF);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= static_cast<uint64_t>(1) << 46;  // descriptor version for sm_100
  d |= static_cast<uint64_t>(2) << 61;  // SWIZZLE_128B
  return d;
}

// 16 lanes x 64 columns of fp32 from TMEM: r[4j+e] = row (lane/4 + 8*(e>>1)), column 8j + 2*(lane%4) + (e&1)
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, float (&r)[32]) {
  uint32_t* u = reinterpret_cast<uint32_t*>(r);
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x8.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]),
        "=r"(u[8]), "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15]),
        "=r"(u[16]), "=r"(u[17]), "=r"(u[18]), "=r"(u[19]), "=r"(u[20]), "=r"(u[21]), "=r"(u[22]), "=r"(u[23]),
        "=r"(u[24]), "=r"(u[25]), "=r"(u[26]), "=r"(u[27]), "=r"(u[28]), "=r"(u[29]), "=r"(u[30]), "=r"(u[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st64(uint32_t taddr, const float (&r)[32]) {
  const uint32_t* u = reinterpret_cast<const uint32_t*>(r);
  asm volatile(
      "tcgen05.st.sync.aligned.16x256b.x8.b32 [%32], "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31};"
      ::"r"(u[0]), "r"(u[1]), "r"(u[2]), "r"(u[3]), "r"(u[4]), "r"(u[5]), "r"(u[6]), "r"(u[7]),
        "r"(u[8]), "r"(u[9]), "r"(u[10]), "r"(u[11]), "r"(u[12]), "r"(u[13]), "r"(u[14]), "r"(u[15]),
        "r"(u[16]), "r"(u[17]), "r"(u[18]), "r"(u[19]), "r"(u[20]), "r"(u[21]), "r"(u[22]), "r"(u[23]),
        "r"(u[24]), "r"(u[25]), "r"(u[26]), "r"(u[27]), "r"(u[28]), "r"(u[29]), "r"(u[30]), "r"(u[31]),
        "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

struct Barriers {
  uint32_t full_k[kStages], full_v[kStages], empty[kStages];
  uint32_t s_full[2], s_free[2];
  uint32_t p_full, pv_done, q_full;
};

}  // namespace tc

using namespace tc;

__global__ void __launch_bounds__(kThreads, 1)
tree_attn_tc_kernel(const AttnParams p, const __grid_constant__ CUtensorMap map_q,
                    const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v) {
  extern __shared__ unsigned char smem_raw[];
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();

  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (base - raw);

  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int T = p.T;

  Barriers bar;
  {
    uint32_t a = base + kOffBar;
    for (int s = 0; s < kStages; ++s) { bar.full_k[s] = a; a += 8; }
    for (int s = 0; s < kStages; ++s) { bar.full_v[s] = a; a += 8; }
    for (int s = 0; s < kStages; ++s) { bar.empty[s] = a; a += 8; }
    bar.s_full[0] = a; a += 8; bar.s_full[1] = a; a += 8;
    bar.s_free[0] = a; a += 8; bar.s_free[1] = a; a += 8;
    bar.p_full = a; a += 8; bar.pv_done = a; a += 8; bar.q_full = a; a += 8;
  }
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kOffMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffMisc + 8);

  // ---- sequence geometry (tiles are anchored at the end of the sequence)
  int P = p.prefix_len[b];
  int n_keys = P + T;
  if (P < 0 || n_keys > p.S_cap) {
    if (threadIdx.x == 0 && split == 0 && h == 0 && p.status != nullptr)
      atomicOr(p.status, SPECVLM_STATUS_BAD_PREFIX);
    P = 0;
    n_keys = 0;
  }
  const int tiles_total = (n_keys + kTile - 1) / kTile;
  const int tps = (tiles_total + p.splits - 1) / p.splits;
  const int tile_begin = min(split * tps, tiles_total);  // tile index counted from the end
  const int n_tiles = min(tile_begin + tps, tiles_total) - tile_begin;

  // ---- set-up: barriers, TMEM
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar.full_k[s], 1);
      mbar_init(bar.full_v[s], 1);
      mbar_init(bar.empty[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar.s_full[i], 1);
      mbar_init(bar.s_free[i], 128);
    }
    mbar_init(bar.p_full, 128);
    mbar_init(bar.pv_done, 1);
    mbar_init(bar.q_full, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // softmax-warp state that outlives the main loop
  float o[16][4];
  float mu0 = -INFINITY, mu1 = -INFINITY, l0 = 0.f, l1 = 0.f;
#pragma unroll
  for (int i = 0; i < 16; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  const int sw = warp - kSoftmaxWarp0;       // 0..3 for softmax warps
  const int quad = warp & 3;                 // TMEM lane quadrant this warp may access
  const int g = lane >> 2, t4 = lane & 3;
  const int row0 = quad * 16 + g, row1 = row0 + 8;

  if (warp == 0) {
    // ======================= TMA producer =======================
    if (lane == 0 && n_tiles > 0) {
      mbar_expect_tx(bar.q_full, kQBytes);
      tma_load_4d(base + kOffQ, &map_q, bar.q_full, 0, 0, h, b);
      tma_load_4d(base + kOffQ + kQBytes / 2, &map_q, bar.q_full, 64, 0, h, b);
      int issued = 0;
      for (int i = 0; i < n_tiles; ++i) {
        const int s = i % kStages;
        if (i >= kStages && !mbar_wait(bar.empty[s], ((i / kStages) & 1) ^ 1, abort_flag)) break;
        const int key0 = n_keys - (tile_begin + i + 1) * kTile;  // may be negative: zero-filled
        const uint32_t sk = base + kOffStage + s * kStageBytes, sv = sk + kKBytes;
        mbar_expect_tx(bar.full_k[s], kKBytes);
        tma_load_4d(sk, &map_k, bar.full_k[s], 0, key0, h, b);
        tma_load_4d(sk + kKBytes / 2, &map_k, bar.full_k[s], 64, key0, h, b);
        mbar_expect_tx(bar.full_v[s], kVBytes);
        tma_load_4d(sv, &map_v, bar.full_v[s], 0, key0, h, b);
        tma_load_4d(sv + kVBytes / 2, &map_v, bar.full_v[s], 64, key0, h, b);
        ++issued;
      }
      if (*abort_flag) {
        // give copies that are still in flight a bounded time to land before the CTA exits
        mbar_wait(bar.q_full, 0, abort_flag);
        for (int i = max(0, issued - kStages); i < issued; ++i) {
          uint32_t spins = 0;
          while (!mbar_try_wait(bar.full_k[i % kStages], (i / kStages) & 1) && ++spins < kSpinLimit) {}
          spins = 0;
          while (!mbar_try_wait(bar.full_v[i % kStages], (i / kStages) & 1) && ++spins < kSpinLimit) {}
        }
      }
    }
  } else if (warp == 1) {
    // ======================= MMA issuer =======================
    if (lane == 0 && n_tiles > 0) {
      constexpr uint32_t idesc_qk = make_idesc(false), idesc_pv = make_idesc(true);
      const uint32_t tmem_o = tmem_base + kColO;
      bool ok = mbar_wait(bar.q_full, 0, abort_flag);
      auto issue_qk = [&](int i) {
        const int s = i % kStages;
        const uint32_t sk = base + kOffStage + s * kStageBytes;
        const uint32_t tmem_s = tmem_base + ((i & 1) ? kColS1 : kColS0);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint64_t ad = make_desc(base + kOffQ + (ks >> 2) * (kQBytes / 2) + (ks & 3) * 32, 16, 1024);
          const uint64_t bd = make_desc(sk + (ks >> 2) * (kKBytes / 2) + (ks & 3) * 32, 16, 1024);
          tc_mma(tmem_s, ad, bd, idesc_qk, ks > 0 ? 1u : 0u);
        }
        tc_commit(bar.s_full[i & 1]);
      };
      if (ok) ok = mbar_wait(bar.full_k[0], 0, abort_flag);
      if (ok) {
        tc_fence_after();
        issue_qk(0);
      }
      for (int i = 0; ok && i < n_tiles; ++i) {
        const int s = i % kStages;
        if (i + 1 < n_tiles) {
          const int s1 = (i + 1) % kStages;
          ok = mbar_wait(bar.full_k[s1], ((i + 1) / kStages) & 1, abort_flag);
          if (ok && i + 1 >= 2) ok = mbar_wait(bar.s_free[(i + 1) & 1], (((i + 1) >> 1) & 1) ^ 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          issue_qk(i + 1);
        }
        ok = mbar_wait(bar.full_v[s], (i / kStages) & 1, abort_flag);
        if (ok) ok = mbar_wait(bar.p_full, i & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sv = base + kOffStage + s * kStageBytes + kKBytes;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint64_t ad = make_desc(base + kOffP + (ks >> 2) * (kPBytes / 2) + (ks & 3) * 32, 16, 1024);
          const uint64_t bd = make_desc(sv + ks * 2048, kVBytes / 2, 1024);
          tc_mma(tmem_o, ad, bd, idesc_pv, (i > 0 || ks > 0) ? 1u : 0u);
        }
        tc_commit(bar.empty[s]);
        tc_commit(bar.pv_done);
      }
    }
  } else {
    // ======================= softmax warps =======================
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
          for (int step = 0; step < kRows && n >= 0 && n < T; ++step) {
            bits |= 1ull << n;
            const int up = par[n];
            n = (up < n) ? up : -1;
          }
        }
        if (pass) mask1 = bits; else mask0 = bits;
      }
    }
    const uint32_t lane_base = static_cast<uint32_t>(quad * 32) << 16;
    bool ok = true;
    for (int i = 0; i < n_tiles && ok; ++i) {
      const int key0 = n_keys - (tile_begin + i + 1) * kTile;
      ok = mbar_wait(bar.s_full[i & 1], (i >> 1) & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      float s[2][32];
      const uint32_t ts = tmem_base + lane_base + ((i & 1) ? kColS1 : kColS0);
      tmem_ld64(ts, s[0]);
      tmem_ld64(ts + 64, s[1]);
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(bar.s_free[i & 1]);

      // scale (log2 domain) and mask: key >= 0; prefix keys visible; tree slot t visible iff mask bit t
      const bool need_mask = (key0 < 0) || (key0 + kTile > P);
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float x = s[hf][4 * j + e] * p.scale_log2;
            if (need_mask) {
              const int key = key0 + hf * 64 + j * 8 + t4 * 2 + (e & 1);
              const uint64_t mw = (e & 2) ? mask1 : mask0;
              const int t = key - P;
              const bool vis = (key >= 0) && ((t < 0) || ((mw >> (t & 63)) & 1ull));
              x = vis ? x : -INFINITY;
            }
            s[hf][4 * j + e] = x;
            if (e & 2) mx1 = fmaxf(mx1, x); else mx0 = fmaxf(mx0, x);
          }
        }
      }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));

      // lazy rescale: the reference maximum only moves when the tile maximum exceeds it by > 2^8
      const bool need0 = (mx0 > mu0 + kRescaleThreshold) || (mu0 == -INFINITY && mx0 > -INFINITY);
      const bool need1 = (mx1 > mu1 + kRescaleThreshold) || (mu1 == -INFINITY && mx1 > -INFINITY);
      const bool any_rescale = __any_sync(0xffffffffu, need0 || need1);

      // P is single-buffered and O is about to be touched: the previous PV must be complete
      if (i > 0) {
        ok = mbar_wait(bar.pv_done, (i - 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
      }
      if (any_rescale) {
        const float a0 = need0 ? exp2f(mu0 - mx0) : 1.f;  // exp2(-inf) = 0 for a row's first visible key
        const float a1 = need1 ? exp2f(mu1 - mx1) : 1.f;
        if (need0) { mu0 = mx0; l0 *= a0; }
        if (need1) { mu1 = mx1; l1 *= a1; }
        if (i > 0) {
          const uint32_t to = tmem_base + lane_base + kColO;
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
            float ov[32];
            tmem_ld64(to + hf * 64, ov);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              ov[4 * j + 0] *= a0; ov[4 * j + 1] *= a0; ov[4 * j + 2] *= a1; ov[4 * j + 3] *= a1;
            }
            tmem_st64(to + hf * 64, ov);
          }
          tmem_wait_st();
        }
      }
      const float ms0 = (mu0 == -INFINITY) ? 0.f : mu0;
      const float ms1 = (mu1 == -INFINITY) ? 0.f : mu1;

      // exponentials, row sums, P as the K-major swizzled A operand: row r, key c ->
      // atom c/64, byte r*128 + (((c%64)/8) ^ (r&7))*16 + (c%8)*2
      float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float p0 = exp2f(s[hf][4 * j + 0] - ms0), p1 = exp2f(s[hf][4 * j + 1] - ms0);
          const float p2 = exp2f(s[hf][4 * j + 2] - ms1), p3 = exp2f(s[hf][4 * j + 3] - ms1);
          sum0 += p0 + p1;
          sum1 += p2 + p3;
          unsigned char* atom = smem + kOffP + hf * (kPBytes / 2);
          *reinterpret_cast<uint32_t*>(atom + row0 * 128 + ((j ^ (row0 & 7)) << 4) + t4 * 4) = pack_bf16(p0, p1);
          *reinterpret_cast<uint32_t*>(atom + row1 * 128 + ((j ^ (row1 & 7)) << 4) + t4 * 4) = pack_bf16(p2, p3);
        }
      }
      l0 += sum0;
      l1 += sum1;
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> tensor-core reads
      tc_fence_before();
      mbar_arrive(bar.p_full);
    }
    // ---- O out of TMEM
    if (ok && n_tiles > 0) {
      ok = mbar_wait(bar.pv_done, (n_tiles - 1) & 1, abort_flag);
      if (ok) {
        tc_fence_after();
        const uint32_t to = tmem_base + lane_base + kColO;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          float ov[32];
          tmem_ld64(to + hf * 64, ov);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            o[hf * 8 + j][0] = ov[4 * j + 0]; o[hf * 8 + j][1] = ov[4 * j + 1];
            o[hf * 8 + j][2] = ov[4 * j + 2]; o[hf * 8 + j][3] = ov[4 * j + 3];
          }
        }
      }
    }
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  }

  // ---- all roles meet; from here on shared-memory stages and TMEM are no longer in use
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const bool aborted = *abort_flag != 0;
  if (aborted && threadIdx.x == 0 && p.status != nullptr) atomicOr(p.status, SPECVLM_STATUS_TIMEOUT);
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }

  uint16_t* obase = p.out + b * p.o_sb + h * p.o_sh;
  if (p.splits == 1) {
    if (warp >= kSoftmaxWarp0 && !aborted) {
      const float i0 = l0 > 0.f ? 1.f / l0 : 0.f, i1 = l1 > 0.f ? 1.f / l1 : 0.f;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int col = i * 8 + t4 * 2;
        if (row0 < T) *reinterpret_cast<uint32_t*>(obase + row0 * p.o_st + col) = pack_bf16(o[i][0] * i0, o[i][1] * i0);
        if (row1 < T) *reinterpret_cast<uint32_t*>(obase + row1 * p.o_st + col) = pack_bf16(o[i][2] * i1, o[i][3] * i1);
      }
    }
    return;
  }

  // ---- partial into this CTA's shared memory, then combine across the cluster through DSMEM
  float* so = reinterpret_cast<float*>(smem + kOffStage);  // [64][128] fp32
  float* sml = so + kRows * kD;                            // [64][2]  (running max, running sum)
  if (warp >= kSoftmaxWarp0) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      *reinterpret_cast<float2*>(so + row0 * kD + i * 8 + t4 * 2) = make_float2(o[i][0], o[i][1]);
      *reinterpret_cast<float2*>(so + row1 * kD + i * 8 + t4 * 2) = make_float2(o[i][2], o[i][3]);
    }
    if (t4 == 0) {
      *reinterpret_cast<float2*>(sml + row0 * 2) = make_float2(mu0, l0);
      *reinterpret_cast<float2*>(sml + row1 * 2) = make_float2(mu1, l1);
    }
  }
  cluster.sync();
  if (warp >= kSoftmaxWarp0 && !aborted) {
    const int nsplit = p.splits;
    int nth = 0;
    for (int row = split; row < T; row += nsplit, ++nth) {
      if ((nth & 3) != sw) continue;
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
  }
  cluster.sync();  // nobody leaves while its shared memory may still be read
}

// ------------------------------------------------------------------ host side

namespace {

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                              CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn encode_fn() {
  static EncodeFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeFn>(ptr);
  });
  return fn;
}

// 4-D bf16 map over [dim3][dim2][rows][128] with element strides; box = 64 elements x box_rows rows.
int make_map(CUtensorMap* map, const void* base, int rows, int dim2, int dim3, int64_t stride_row,
             int64_t stride2, int64_t stride3, int box_rows) {
  const cuuint64_t dims[4] = {static_cast<cuuint64_t>(tc::kD), static_cast<cuuint64_t>(rows),
                              static_cast<cuuint64_t>(dim2), static_cast<cuuint64_t>(dim3)};
  // a stride of 0 (size-1 dimension) is not accepted by the encoder: any positive multiple of 16 works there
  auto fix = [&](int64_t s, int64_t fallback) { return static_cast<cuuint64_t>((s > 0 ? s : fallback) * 2); };
  const cuuint64_t strides[3] = {fix(stride_row, tc::kD), fix(stride2, static_cast<int64_t>(rows) * tc::kD),
                                 fix(stride3, static_cast<int64_t>(rows) * tc::kD * dim2)};
  const cuuint32_t box[4] = {64, static_cast<cuuint32_t>(box_rows), 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = encode_fn()(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box,
                           estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(SPECVLM_ERR_CUDA, "cuTensorMapEncodeTiled failed with code " + std::to_string(r));
  return SPECVLM_OK;
}

}  // namespace

bool attn_tc_available() { return encode_fn() != nullptr; }

int launch_attn_tc(const AttnParams& p, const specvlm_attn_desc& d, cudaStream_t stream) {
  if (!attn_tc_available()) return fail(SPECVLM_ERR_UNSUPPORTED, "tensor-map encoder not available from the driver");
  CUtensorMap mq, mk, mv;
  int rc = make_map(&mq, p.q, d.T, d.H, d.B, d.q_stride_t, d.q_stride_h, d.q_stride_b, tc::kRows);
  if (rc == SPECVLM_OK) rc = make_map(&mk, p.k, d.S_cap, d.H, d.B, d.k_stride_s, d.k_stride_h, d.k_stride_b, tc::kTile);
  if (rc == SPECVLM_OK) rc = make_map(&mv, p.v, d.S_cap, d.H, d.B, d.v_stride_s, d.v_stride_h, d.v_stride_b, tc::kTile);
  if (rc != SPECVLM_OK) return rc;

  static bool attr_set[64] = {};
  int dev = 0;
  rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice");
  if (rc != SPECVLM_OK) return rc;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    rc = check_cuda(cudaFuncSetAttribute(tree_attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         tc::kSmemBytes),
                    "attn (tcgen05) smem attribute");
    if (rc != SPECVLM_OK) return rc;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.splits, d.H, d.B);
  cfg.blockDim = dim3(tc::kThreads);
  cfg.dynamicSmemBytes = tc::kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = p.splits;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return check_cuda(cudaLaunchKernelEx(&cfg, tree_attn_tc_kernel, p, mq, mk, mv), "tree_verify_attn (tcgen05) launch");
}

}  // namespace specvlm
