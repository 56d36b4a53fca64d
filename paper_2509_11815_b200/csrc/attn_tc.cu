// Tree-verification attention on the Blackwell tensor path (sm_100a): tcgen05.mma with TMEM
// accumulators, TMA-staged K/V tiles, warp-specialised roles, cluster/DSMEM split combine,
// programmatic dependent launch.
//
// What it computes: tree attention of the <= 64 draft-tree queries over the KV prefix plus the
// tree's own slots (Sections 3.1, 4.1), streaming the KV cache once from HBM (Section 3.2).
//
// One CTA per (sequence, head, split); the splits of one (sequence, head) are one thread-block
// cluster. A CTA uses less than half of an SM (about 105 KB of shared memory, 256 TMEM columns),
// so the CTAs of the next launch can become resident while this launch drains.
// Roles inside a CTA (192 threads):
//   warp 0      TMA producer: Q once, then 64-key K tiles (ring of 3) and V tiles (ring of 2), one
//               5-D cp.async.bulk.tensor per tile, 128-byte swizzle, no multicast; owns the TMEM
//               allocation
//   warp 1      one lane issues tcgen05.mma: S = Q K^T (M=64, N=64, K=16 x 8) into one of two TMEM
//               buffers, O += P V (M=64, N=128, K=16 x 4); tcgen05.commit signals the mbarriers
//   warps 2..5  softmax: tcgen05.ld of their 16 rows of S, tree mask as one 64-bit visibility word
//               per row and tile, running max with a lazy rescale of O in TMEM, exp2, bf16 P
//               written to shared memory in the K-major swizzled operand layout
// Key tiles are anchored at the END of the sequence (tile j covers keys [n - 64 (j+1), n - 64 j)),
// so the tree slots always fall in tile 0, the lowest tile may start at a negative key index,
// which TMA fills with zeros, and no tile contains a cache slot beyond prefix + T: uninitialised
// slots are never loaded. A CTA walks its tiles from low keys to high keys, so the tile with the
// tree slots comes last.
// Every mbarrier wait is bounded; a wait that gives up sets SPECVLM_STATUS_TIMEOUT, the CTA still
// reaches the cluster barriers, frees its TMEM and returns.
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
constexpr int kThreads = 192;
constexpr int kSoftmaxWarp0 = 2;
constexpr uint32_t kSpinLimit = 1u << 22;      // polls of a possibly suspending try_wait
constexpr uint32_t kPollLimit = 1u << 25;      // turns of a non-blocking polling loop (well under a second)
constexpr float kRescaleThreshold = 8.0f;  // log2 units; P stays <= 2^8
constexpr int kLandStride = kD + 4;        // floats per exchange row: 128 values, (max, sum), padding

// Two configurations of the same kernel:
//   throughput: 64-key tiles, K ring 3 / V ring 2, half an SM per CTA (two CTAs per SM, so the next
//               launch can become resident while this one drains)
//   latency   : 128-key tiles, K ring 3 / V ring 3, a whole SM per CTA (deepest prefetch for one launch)
template <int TILE_, int KS_, int VS_, int MINB_>
struct Cfg {
  static constexpr int kTile = TILE_;         // keys per tile
  static constexpr int kKStages = KS_;
  static constexpr int kVStages = VS_;
  static constexpr int kMinBlocks = MINB_;
  static constexpr int kHalves = TILE_ / 64;  // 64-key swizzle atoms per tile
  // shared memory map (offsets from a 1024-byte aligned base)
  static constexpr int kQBytes = kRows * kD * 2;      // two 64x64 swizzle atoms (d halves)
  static constexpr int kPBytes = kRows * TILE_ * 2;   // kHalves 64x64 swizzle atoms
  static constexpr int kKBytes = TILE_ * kD * 2;      // two TILE-row x 128-byte boxes (d halves)
  static constexpr int kVBytes = TILE_ * kD * 2;
  static constexpr int kOffQ = 0;
  static constexpr int kOffP = kOffQ + kQBytes;
  static constexpr int kOffK = kOffP + kPBytes;
  static constexpr int kOffV = kOffK + KS_ * kKBytes;
  static constexpr int kOffBar = kOffV + VS_ * kVBytes;
  static constexpr int kNumBars = 2 * KS_ + 2 * VS_ + 2 + 2 + 1 + 1 + 1 + 1;
  static constexpr int kOffMisc = kOffBar + kNumBars * 8;
  static constexpr int kSmemBytes = kOffMisc + 64 + 1024;  // + alignment slack
  static_assert(kSmemBytes <= (MINB_ == 2 ? 115712 : 232448), "shared memory budget");
  // staging + landing zones of the split exchange: 2 * ns * ceil(64/ns) rows (worst case ns = 7)
  static_assert(2 * 7 * 10 * kLandStride * 4 <= KS_ * kKBytes + VS_ * kVBytes, "exchange zones");
  // TMEM columns: S0 [0,TILE), S1 [TILE,2 TILE), O [2 TILE, 2 TILE + 128)
  static constexpr uint32_t kTmemCols = TILE_ == 64 ? 256 : 512;
  static constexpr uint32_t kColS0 = 0, kColS1 = TILE_, kColO = 2 * TILE_;
};
using CfgThroughput = Cfg<64, 3, 2, 2>;
using CfgLatency = Cfg<128, 3, 3, 1>;

// tcgen05 instruction descriptor, kind::f16: fp32 accumulate, bf16 A and B, K-major A, M = 64
constexpr uint32_t make_idesc(uint32_t n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((n >> 3) << 17) | ((64u >> 4) << 24);
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
// Non-blocking poll. mbarrier.try_wait may suspend the thread for a system-dependent time when the
// phase is not complete; the producer and the MMA issuer poll several barriers in turn and must
// not sleep on one while another is ready, so they use test_wait.
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false after kSpinLimit unsuccessful polls or once another role has given up.
__device__ __noinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 1023u) == 1023u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

// ---- TMA
// One copy brings both 64-column halves of `rows x 128` bf16 (coordinates: column 0, row, half 0,
// head, sequence); the halves land one after the other, each as rows of 128 swizzled bytes.
__device__ __forceinline__ void tma_load_rows(uint32_t dst, const CUtensorMap* map, uint32_t bar, int row, int h,
                                              int b) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %3, %5, %6}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(0), "r"(row), "r"(h), "r"(b)
      : "memory");
}

// ---- programmatic dependent launch
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

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
// 16 lanes x 32 columns: r[4j+e], j = 0..3
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&r)[16]) {
  uint32_t* u = reinterpret_cast<uint32_t*>(r);
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x4.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]),
        "=r"(u[8]), "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&r)[16]) {
  const uint32_t* u = reinterpret_cast<const uint32_t*>(r);
  asm volatile(
      "tcgen05.st.sync.aligned.16x256b.x4.b32 [%16], {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};"
      ::"r"(u[0]), "r"(u[1]), "r"(u[2]), "r"(u[3]), "r"(u[4]), "r"(u[5]), "r"(u[6]), "r"(u[7]),
        "r"(u[8]), "r"(u[9]), "r"(u[10]), "r"(u[11]), "r"(u[12]), "r"(u[13]), "r"(u[14]), "r"(u[15]),
        "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 2^x; -inf -> 0
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

// Address of the same shared-memory offset in the CTA of rank `rank` of this cluster.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_addr, int rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_cluster_f32x2(uint32_t addr, float a, float b) {
  asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(addr), "f"(a), "f"(b) : "memory");
}

}  // namespace tc

using namespace tc;

template <class C>
__global__ void __launch_bounds__(kThreads, C::kMinBlocks)
tree_attn_tc_kernel(const AttnParams p, const __grid_constant__ CUtensorMap map_q,
                    const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v) {
  constexpr int kTile = C::kTile, kKStages = C::kKStages, kVStages = C::kVStages, kHalves = C::kHalves;
  constexpr int kQBytes = C::kQBytes, kKBytes = C::kKBytes, kVBytes = C::kVBytes;
  constexpr int kOffQ = C::kOffQ, kOffP = C::kOffP, kOffK = C::kOffK, kOffV = C::kOffV, kOffBar = C::kOffBar;
  constexpr int kNumBars = C::kNumBars, kOffMisc = C::kOffMisc;
  constexpr uint32_t kTmemCols = C::kTmemCols, kColS0 = C::kColS0, kColS1 = C::kColS1, kColO = C::kColO;
  extern __shared__ unsigned char smem_raw[];
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();

  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (base - raw);

  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int T = p.T;

  // barrier addresses: full_k[] empty_k[] full_v[] empty_v[] s_full[2] s_free[2] p_full pv_done q_full land_full
  const uint32_t bar0 = base + kOffBar;
  auto FULL_K = [&](int s) { return bar0 + 8u * s; };
  auto EMPTY_K = [&](int s) { return bar0 + 8u * (kKStages + s); };
  auto FULL_V = [&](int s) { return bar0 + 8u * (2 * kKStages + s); };
  auto EMPTY_V = [&](int s) { return bar0 + 8u * (2 * kKStages + kVStages + s); };
  const uint32_t bar1 = bar0 + 8u * (2 * kKStages + 2 * kVStages);
  auto S_FULL = [&](int i) { return bar1 + 8u * i; };
  auto S_FREE = [&](int i) { return bar1 + 8u * (2 + i); };
  const uint32_t P_FULL = bar1 + 32, PV_DONE = bar1 + 40, Q_FULL = bar1 + 48, LAND_FULL = bar1 + 56;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kOffMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffMisc + 8);

  const bool inputs_stable = (p.flags & SPECVLM_ATTN_FLAG_INPUTS_STABLE) != 0;
  const bool prefix_stable = inputs_stable || (p.flags & SPECVLM_ATTN_FLAG_PREFIX_STABLE) != 0;
  // With either promise prefix_len is not written by the preceding kernel: its load is issued
  // first, so that its latency runs beside the set-up below instead of after it.
  int prefix_raw = prefix_stable ? p.prefix_len[b] : 0;

  // ---- set-up that touches no global input: tensor-map prefetch, barriers, TMEM
  if (threadIdx.x == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_k)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_v)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_q)) : "memory");
    for (int i = 0; i < kNumBars; ++i) mbar_init(bar0 + 8u * i, 1);
    mbar_init(S_FREE(0), 128);
    mbar_init(S_FREE(1), 128);
    mbar_init(P_FULL, 128);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // Without a promise from the caller, nothing below may run before the preceding kernel has
  // completed. Only then is the next launch allowed to start: a successor that was promised stable
  // inputs must not overtake work that this kernel itself still had to wait for.
  if (!prefix_stable) {
    pdl_wait();
    prefix_raw = p.prefix_len[b];
    pdl_launch_dependents();
  } else if (inputs_stable) {
    pdl_launch_dependents();  // this launch never waits before it reads
  }
  // PREFIX_STABLE alone: the producer lets the next launch start once its own wait is over
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // ---- sequence geometry
  int P = prefix_raw;
  int n_keys = P + T;
  if (P < 0 || n_keys > p.S_cap) {
    if (threadIdx.x == 0 && split == 0 && h == 0 && p.status != nullptr)
      atomicOr(p.status, SPECVLM_STATUS_BAD_PREFIX);
    P = 0;
    n_keys = 0;
  }
  const int tiles_total = (n_keys + kTile - 1) / kTile;
  const int tps = (tiles_total + p.splits - 1) / p.splits;
  const int tile_begin = min(split * tps, tiles_total);  // tile index counted from the end of the sequence
  const int n_tiles = min(tile_begin + tps, tiles_total) - tile_begin;
  // step i of this CTA works on tile (tile_begin + n_tiles - 1 - i): low keys first, tree slots last
  auto KEY0 = [&](int i) { return n_keys - (tile_begin + n_tiles - i) * kTile; };

  const int sw = warp - kSoftmaxWarp0;  // 0..3 for softmax warps
  const int quad = warp & 3;            // TMEM lane quadrant this warp may access
  const int g = lane >> 2, t4 = lane & 3;
  const int row0 = quad * 16 + g, row1 = row0 + 8;
  const uint32_t lane_base = static_cast<uint32_t>(quad * 32) << 16;
  float mu0 = -INFINITY, mu1 = -INFINITY, l0 = 0.f, l1 = 0.f;

  if (warp == 0) {
    // ======================= TMA producer =======================
    // K and V rings advance independently: a slot is refilled as soon as the MMAs that read it
    // have completed, whichever ring that is.
    if (lane == 0 && n_tiles > 0) {
      auto issue_q = [&]() {
        mbar_expect_tx(Q_FULL, kQBytes);
        tma_load_rows(base + kOffQ, &map_q, Q_FULL, 0, h, b);
      };
      auto issue_k = [&](int i) {
        const int sk = i % kKStages;
        const uint32_t dk = base + kOffK + sk * kKBytes;
        mbar_expect_tx(FULL_K(sk), kKBytes);
        tma_load_rows(dk, &map_k, FULL_K(sk), KEY0(i), h, b);
      };
      auto issue_v = [&](int i) {
        const int sv = i % kVStages;
        const uint32_t dv = base + kOffV + sv * kVBytes;
        mbar_expect_tx(FULL_V(sv), kVBytes);
        tma_load_rows(dv, &map_v, FULL_V(sv), KEY0(i), h, b);
      };
      int ik = 0, iv = 0;
      if (prefix_stable && !inputs_stable) {
        // Pure prefix tiles may be fetched before the preceding kernel has completed; Q, the tree
        // arrays and the tile with the tree slots are read only afterwards.
        while (ik < n_tiles && ik < kKStages && KEY0(ik) + kTile <= P) issue_k(ik++);
        while (iv < n_tiles && iv < kVStages && KEY0(iv) + kTile <= P) issue_v(iv++);
        pdl_wait();
        pdl_launch_dependents();
      }
      issue_q();
      uint32_t idle = 0;
      while (ik < n_tiles || iv < n_tiles) {
        bool progress = false;
        if (ik < n_tiles && (ik < kKStages || mbar_test(EMPTY_K(ik % kKStages), ((ik / kKStages) & 1) ^ 1))) {
          issue_k(ik++);
          progress = true;
        }
        if (iv < n_tiles && (iv < kVStages || mbar_test(EMPTY_V(iv % kVStages), ((iv / kVStages) & 1) ^ 1))) {
          issue_v(iv++);
          progress = true;
        }
        if (progress) {
          idle = 0;
        } else if (++idle > kPollLimit || ((idle & 1023u) == 0 && *abort_flag)) {
          *abort_flag = 1;
          break;
        }
      }
      if (*abort_flag) {
        // give copies that are still in flight a bounded time to land before the CTA exits
        for (int i = max(0, ik - kKStages); i < ik; ++i) {
          uint32_t spins = 0;
          while (!mbar_try_wait(FULL_K(i % kKStages), (i / kKStages) & 1) && ++spins < kSpinLimit) {}
        }
        for (int i = max(0, iv - kVStages); i < iv; ++i) {
          uint32_t spins = 0;
          while (!mbar_try_wait(FULL_V(i % kVStages), (i / kVStages) & 1) && ++spins < kSpinLimit) {}
        }
      }
    }
  } else if (warp == 1) {
    // ======================= MMA issuer =======================
    if (lane == 0 && n_tiles > 0) {
      constexpr uint32_t idesc_qk = make_idesc(kTile, false), idesc_pv = make_idesc(kD, true);
      const uint32_t tmem_o = tmem_base + kColO;
      // This one thread issues every MMA, and a lone thread issues a dependent instruction only
      // every few cycles, so the per-MMA instruction count matters. Matrix descriptors of one
      // operand buffer differ only in their start-address field (byte address >> 4, 14 bits, and
      // shared-memory addresses stay below 2^18): one descriptor per buffer is built up front and
      // moving it is one addition. Ring stages and barrier parities are carried along instead of
      // being recomputed with divisions.
      const uint64_t q_desc = make_desc(base + kOffQ, 16, 1024);
      const uint64_t p_desc = make_desc(base + kOffP, 16, 1024);
      const uint64_t k_desc0 = make_desc(base + kOffK, 16, 1024);
      const uint64_t v_desc0 = make_desc(base + kOffV, kVBytes / 2, 1024);
      int k_stage = 0, v_stage = 0;         // ring stage of the next S = Q K^T / the next O += P V
      uint32_t k_parity = 0, v_parity = 0;  // parity of that stage's "full" barrier
      auto issue_qk = [&](int i) {
        const uint64_t kd = k_desc0 + static_cast<uint64_t>(k_stage * (kKBytes >> 4));
        const uint32_t tmem_s = tmem_base + ((i & 1) ? kColS1 : kColS0);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint64_t ad = q_desc + static_cast<uint64_t>(((ks >> 2) * (kQBytes / 2) + (ks & 3) * 32) >> 4);
          const uint64_t bd = kd + static_cast<uint64_t>(((ks >> 2) * (kKBytes / 2) + (ks & 3) * 32) >> 4);
          tc_mma(tmem_s, ad, bd, idesc_qk, ks > 0 ? 1u : 0u);
        }
        tc_commit(EMPTY_K(k_stage));  // K stage free once these MMAs have read it
        tc_commit(S_FULL(i & 1));
        if (++k_stage == kKStages) { k_stage = 0; k_parity ^= 1u; }
      };
      auto issue_pv = [&](int i) {
        const uint64_t vd = v_desc0 + static_cast<uint64_t>(v_stage * (kVBytes >> 4));
#pragma unroll
        for (int ks = 0; ks < kTile / 16; ++ks) {
          const uint64_t ad = p_desc + static_cast<uint64_t>(((ks >> 2) * 8192 + (ks & 3) * 32) >> 4);
          const uint64_t bd = vd + static_cast<uint64_t>((ks * 2048) >> 4);
          tc_mma(tmem_o, ad, bd, idesc_pv, (i > 0 || ks > 0) ? 1u : 0u);
        }
        tc_commit(EMPTY_V(v_stage));
        tc_commit(PV_DONE);
        if (++v_stage == kVStages) { v_stage = 0; v_parity ^= 1u; }
      };
      // Whichever of "O += P V of tile ip" and "S = Q K^T of tile iq" has its operands ready is
      // issued; PV is looked at first because the softmax warps wait for its completion.
      bool ok = mbar_wait(Q_FULL, 0, abort_flag);
      int iq = 0, ip = 0;
      uint32_t idle = 0;
      while (ok && ip < n_tiles) {
        bool progress = false;
        if (ip < iq && mbar_test(P_FULL, ip & 1) && mbar_test(FULL_V(v_stage), v_parity)) {
          tc_fence_after();
          issue_pv(ip++);
          progress = true;
        }
        if (iq < n_tiles && iq < ip + 2 && mbar_test(FULL_K(k_stage), k_parity) &&
            (iq < 2 || mbar_test(S_FREE(iq & 1), ((iq >> 1) & 1) ^ 1))) {
          tc_fence_after();
          issue_qk(iq++);
          progress = true;
        }
        if (progress) {
          idle = 0;
        } else if (++idle > kPollLimit || ((idle & 1023u) == 0 && *abort_flag)) {
          *abort_flag = 1;
          ok = false;
        }
      }
    }
  } else {
    // ======================= softmax warps =======================
    if (prefix_stable && !inputs_stable) pdl_wait();  // the tree arrays may come from the preceding kernel
    uint64_t mask0 = 0, mask1 = 0;
    if (p.mask != nullptr) {
      if (row0 < T) mask0 = p.mask[b * T + row0];
      if (row1 < T) mask1 = p.mask[b * T + row1];
    } else {
      const int32_t* par = p.parent + b * T;
#pragma unroll 1
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
    const uint64_t tmask = (T >= 64) ? ~0ull : ((1ull << T) - 1ull);
    mask0 &= tmask;
    mask1 &= tmask;
    unsigned char* prow0 = smem + kOffP + row0 * 128 + t4 * 4;
    unsigned char* prow1 = prow0 + 8 * 128;
    bool ok = true;
#pragma unroll 1
    for (int i = 0; i < n_tiles && ok; ++i) {
      const int key0 = KEY0(i);
      // visibility of the tile's columns (bit c of half hf <-> key key0 + 64 hf + c), shifted to this
      // thread's column pair: columns [a, d) are prefix keys, column d + t is tree slot t
      uint64_t vis0[kHalves], vis1[kHalves];
      {
        const int a = key0 < 0 ? -key0 : 0;
        const int d = P - key0;
#pragma unroll
        for (int hf = 0; hf < kHalves; ++hf) {
          const int lo = max(a - 64 * hf, 0), hi = min(d - 64 * hf, 64);
          uint64_t pre = 0;
          if (hi > lo) pre = ((~0ull) >> (64 - (hi - lo))) << lo;
          const int sh = d - 64 * hf;  // column of tree slot 0 in this half
          uint64_t t0 = 0, t1 = 0;
          if (sh >= 0 && sh < 64) { t0 = mask0 << sh; t1 = mask1 << sh; }
          else if (sh < 0 && sh > -64) { t0 = mask0 >> (-sh); t1 = mask1 >> (-sh); }
          vis0[hf] = (pre | t0) >> (2 * t4);
          vis1[hf] = (pre | t1) >> (2 * t4);
        }
      }

      ok = mbar_wait(S_FULL(i & 1), (i >> 1) & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      float s[kHalves][32];
#pragma unroll
      for (int hf = 0; hf < kHalves; ++hf)
        tmem_ld64(tmem_base + lane_base + ((i & 1) ? kColS1 : kColS0) + 64 * hf, s[hf]);
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(S_FREE(i & 1));

      // tiles of prefix keys only (the common case) need no masking; the test is uniform over the CTA
      if (key0 < 0 || key0 + kTile > P) {
#pragma unroll
        for (int hf = 0; hf < kHalves; ++hf) {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const bool v = (((e & 2) ? vis1[hf] : vis0[hf]) >> (8 * j + (e & 1))) & 1ull;
              s[hf][4 * j + e] = v ? s[hf][4 * j + e] : -INFINITY;
            }
          }
        }
      }
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int hf = 0; hf < kHalves; ++hf) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          mx0 = fmaxf(mx0, fmaxf(s[hf][4 * j + 0], s[hf][4 * j + 1]));
          mx1 = fmaxf(mx1, fmaxf(s[hf][4 * j + 2], s[hf][4 * j + 3]));
        }
      }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      mx0 *= p.scale_log2;  // scores are compared and exponentiated in the log2 domain; scale > 0
      mx1 *= p.scale_log2;

      // lazy rescale: the reference maximum only moves when the tile maximum exceeds it by > 2^8
      const bool need0 = (mx0 > mu0 + kRescaleThreshold) || (mu0 == -INFINITY && mx0 > -INFINITY);
      const bool need1 = (mx1 > mu1 + kRescaleThreshold) || (mu1 == -INFINITY && mx1 > -INFINITY);
      const bool any_rescale = __any_sync(0xffffffffu, need0 || need1);

      // P is single-buffered and O is about to be touched: the previous PV must be complete
      if (i > 0) {
        ok = mbar_wait(PV_DONE, (i - 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
      }
      if (any_rescale) {
        const float a0 = need0 ? exp2f(mu0 - mx0) : 1.f;  // exp2(-inf) = 0 for a row's first visible key
        const float a1 = need1 ? exp2f(mu1 - mx1) : 1.f;
        if (need0) { mu0 = mx0; l0 *= a0; }
        if (need1) { mu1 = mx1; l1 *= a1; }
        if (i > 0) {
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            const uint32_t to = tmem_base + lane_base + kColO + c * 32;
            float ov[16];
            tmem_ld32(to, ov);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              ov[4 * j + 0] *= a0; ov[4 * j + 1] *= a0; ov[4 * j + 2] *= a1; ov[4 * j + 3] *= a1;
            }
            tmem_st32(to, ov);
          }
          tmem_wait_st();
        }
      }
      const float nm0 = (mu0 == -INFINITY) ? 0.f : -mu0;
      const float nm1 = (mu1 == -INFINITY) ? 0.f : -mu1;

      // exponentials, row sums, P as the K-major swizzled A operand: row r, key c ->
      // atom c/64, byte r*128 + (((c%64)/8) ^ (r&7))*16 + (c%8)*2   (r & 7 == g for both rows)
      float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
      for (int hf = 0; hf < kHalves; ++hf) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float p0 = ex2(fmaf(s[hf][4 * j + 0], p.scale_log2, nm0));
          const float p1 = ex2(fmaf(s[hf][4 * j + 1], p.scale_log2, nm0));
          const float p2 = ex2(fmaf(s[hf][4 * j + 2], p.scale_log2, nm1));
          const float p3 = ex2(fmaf(s[hf][4 * j + 3], p.scale_log2, nm1));
          sum0 += p0 + p1;
          sum1 += p2 + p3;
          const int off = hf * 8192 + ((j ^ g) << 4);
          *reinterpret_cast<uint32_t*>(prow0 + off) = pack_bf16(p0, p1);
          *reinterpret_cast<uint32_t*>(prow1 + off) = pack_bf16(p2, p3);
        }
      }
      l0 += sum0;
      l1 += sum1;
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> tensor-core reads
      tc_fence_before();
      mbar_arrive(P_FULL);
    }
    if (ok && n_tiles > 0) {
      ok = mbar_wait(PV_DONE, (n_tiles - 1) & 1, abort_flag);
      tc_fence_after();
    }
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  }

  uint16_t* obase = p.out + b * p.o_sb + h * p.o_sh;
  const bool have_o = n_tiles > 0;  // otherwise the TMEM accumulator was never written
  const uint32_t to0 = tmem_base + lane_base + kColO;

  if (p.splits == 1) {
    // ---- single split: normalise O straight out of TMEM
    const bool aborted_local = *abort_flag != 0;
    if (warp >= kSoftmaxWarp0 && !aborted_local) {
      if (inputs_stable) pdl_wait();  // `out` may still be in use by the preceding kernel
      const float i0 = l0 > 0.f ? 1.f / l0 : 0.f, i1 = l1 > 0.f ? 1.f / l1 : 0.f;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        float ov[16];
        if (have_o) {
          tmem_ld32(to0 + c * 32, ov);
          tmem_wait_ld();
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) ov[j] = 0.f;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int col = c * 32 + j * 8 + t4 * 2;
          if (row0 < T) *reinterpret_cast<uint32_t*>(obase + row0 * p.o_st + col) = pack_bf16(ov[4 * j] * i0, ov[4 * j + 1] * i0);
          if (row1 < T) *reinterpret_cast<uint32_t*>(obase + row1 * p.o_st + col) = pack_bf16(ov[4 * j + 2] * i1, ov[4 * j + 3] * i1);
        }
      }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (*abort_flag != 0 && threadIdx.x == 0 && p.status != nullptr) atomicOr(p.status, SPECVLM_STATUS_TIMEOUT);
    if (warp == 0)
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    return;
  }

  // ---- exchange through distributed shared memory. Output row r is combined by CTA r % splits.
  // Each CTA first writes its unnormalised O rows (with the row's running max and sum in the
  // row's padding) into a local staging area grouped by owner. After the first cluster barrier
  // every CTA of the cluster is past its main loop, so the K/V rings are free everywhere; one
  // thread then sends each owner its group with one bulk shared-to-shared copy that completes
  // on the owner's mbarrier. A CTA combines its rows once its own landing zone is complete, and
  // leaves after the second cluster barrier, when nobody can still be reading its staging area.
  const int ns = p.splits;
  const int rk = (kRows + ns - 1) / ns;                    // rows per (source, owner) group
  const uint32_t group_bytes = rk * kLandStride * 4;       // multiple of 16
  float* stage = reinterpret_cast<float*>(smem + kOffK);   // [owner][rk][kLandStride]
  const uint32_t stage_u32 = base + kOffK;
  const uint32_t land_u32 = stage_u32 + ns * group_bytes;  // [source][rk][kLandStride]
  const float* landp = stage + ns * rk * kLandStride;
  const bool aborted0 = *abort_flag != 0;
  if (threadIdx.x == 0) mbar_expect_tx(LAND_FULL, (ns - 1) * group_bytes);  // armed before anyone may send
  if (warp >= kSoftmaxWarp0 && !aborted0) {
    // Within a row the 128 values are rotated by 8 columns per owner: the eight rows a warp stores
    // at once then fall into different banks (rows of different owners are a multiple of 32 words
    // apart otherwise). The owner undoes the rotation when it reads.
    const int o0 = row0 % ns, o1 = row1 % ns;
    float* d0 = stage + (o0 * rk + row0 / ns) * kLandStride;
    float* d1 = stage + (o1 * rk + row1 / ns) * kLandStride;
    float ov[4][16];
    if (have_o) {
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32(to0 + c * 32, ov[c]);
      tmem_wait_ld();
    } else {
#pragma unroll
      for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int j = 0; j < 16; ++j) ov[c][j] = 0.f;
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int col = c * 32 + j * 8 + t4 * 2;
        *reinterpret_cast<float2*>(d0 + ((col + 8 * o0) & (kD - 1))) = make_float2(ov[c][4 * j + 0], ov[c][4 * j + 1]);
        *reinterpret_cast<float2*>(d1 + ((col + 8 * o1) & (kD - 1))) = make_float2(ov[c][4 * j + 2], ov[c][4 * j + 3]);
      }
    }
    if (t4 == 0) {
      *reinterpret_cast<float2*>(d0 + kD) = make_float2(mu0, l0);
      *reinterpret_cast<float2*>(d1 + kD) = make_float2(mu1, l1);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // staging is read by the bulk copies
  }
  tc_fence_before();
  cluster.sync();
  tc_fence_after();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
  if (threadIdx.x == kSoftmaxWarp0 * 32) {
    for (int dst = 0; dst < ns; ++dst) {
      if (dst == split) continue;
      asm volatile(
          "cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
          ::"r"(map_to_rank(land_u32 + split * group_bytes, dst)), "r"(stage_u32 + dst * group_bytes),
            "r"(group_bytes), "r"(map_to_rank(LAND_FULL, dst)) : "memory");
    }
  }
  bool landed = true;
  if (warp >= kSoftmaxWarp0) landed = mbar_wait(LAND_FULL, 0, abort_flag);
  cluster.barrier_arrive();
  const bool aborted = *abort_flag != 0;
  if (aborted && threadIdx.x == 0 && p.status != nullptr) atomicOr(p.status, SPECVLM_STATUS_TIMEOUT);
  if (warp >= kSoftmaxWarp0 && !aborted && landed) {
    if (inputs_stable) pdl_wait();  // `out` may still be in use by the preceding kernel
    // A warp pass covers four owned rows (k = sw + 4 rr + 16 pass); lane (rr, cc) combines 16 columns.
    const int rr = lane >> 3, cc = lane & 7;
#pragma unroll 1
    for (int k = sw + 4 * rr; k < rk; k += 16) {
      const int row = split + k * ns;
      if (row < T) {
        // all sources' (max, sum) pairs first, then all value loads: nothing here depends on a
        // previous shared-memory load (at most 8 splits reach this path)
        const float* srcs[8];
        float2 ml[8];
        float mstar = -INFINITY;
#pragma unroll
        for (int s2 = 0; s2 < 8; ++s2) {
          srcs[s2] = (s2 == split ? stage + split * rk * kLandStride : landp + s2 * rk * kLandStride) + k * kLandStride;
          ml[s2] = s2 < ns ? *reinterpret_cast<const float2*>(srcs[s2] + kD) : make_float2(-INFINITY, 0.f);
          mstar = fmaxf(mstar, ml[s2].x);
        }
        float4 acc[4];
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) acc[q4] = make_float4(0.f, 0.f, 0.f, 0.f);
        float lsum = 0.f;
#pragma unroll
        for (int s2 = 0; s2 < 8; ++s2) {
          if (s2 < ns) {
            const float w = (ml[s2].x == -INFINITY) ? 0.f : ex2(ml[s2].x - mstar);
            lsum += w * ml[s2].y;
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
              const float4 x = *reinterpret_cast<const float4*>(srcs[s2] + ((cc * 16 + q4 * 4 + 8 * split) & (kD - 1)));
              acc[q4].x += w * x.x; acc[q4].y += w * x.y; acc[q4].z += w * x.z; acc[q4].w += w * x.w;
            }
          }
        }
        const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
        uint4 lo, hi;
        lo.x = pack_bf16(acc[0].x * inv, acc[0].y * inv); lo.y = pack_bf16(acc[0].z * inv, acc[0].w * inv);
        lo.z = pack_bf16(acc[1].x * inv, acc[1].y * inv); lo.w = pack_bf16(acc[1].z * inv, acc[1].w * inv);
        hi.x = pack_bf16(acc[2].x * inv, acc[2].y * inv); hi.y = pack_bf16(acc[2].z * inv, acc[2].w * inv);
        hi.z = pack_bf16(acc[3].x * inv, acc[3].y * inv); hi.w = pack_bf16(acc[3].z * inv, acc[3].w * inv);
        uint4* dst = reinterpret_cast<uint4*>(obase + row * p.o_st + cc * 16);
        dst[0] = lo;
        dst[1] = hi;
      }
    }
  }
  cluster.barrier_wait();
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

// 5-D bf16 map over [dim3][dim2][rows][2 halves][64] with element strides; box = 64 elements x
// box_rows rows x both halves, so one copy fills a whole operand tile in the layout the 128-byte
// swizzled matrix descriptors expect (half 0 rows, then half 1 rows).
int make_map(CUtensorMap* map, const void* base, int rows, int dim2, int dim3, int64_t stride_row,
             int64_t stride2, int64_t stride3, int box_rows) {
  const cuuint64_t dims[5] = {64, static_cast<cuuint64_t>(rows), 2, static_cast<cuuint64_t>(dim2),
                              static_cast<cuuint64_t>(dim3)};
  // a stride of 0 (size-1 dimension) is not accepted by the encoder: any positive multiple of 16 works there
  auto fix = [&](int64_t s, int64_t fallback) { return static_cast<cuuint64_t>((s > 0 ? s : fallback) * 2); };
  const cuuint64_t strides[4] = {fix(stride_row, tc::kD), 128, fix(stride2, static_cast<int64_t>(rows) * tc::kD),
                                 fix(stride3, static_cast<int64_t>(rows) * tc::kD * dim2)};
  const cuuint32_t box[5] = {64, static_cast<cuuint32_t>(box_rows), 2, 1, 1};
  const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  CUresult r = encode_fn()(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box,
                           estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(SPECVLM_ERR_CUDA, "cuTensorMapEncodeTiled failed with code " + std::to_string(r));
  return SPECVLM_OK;
}

}  // namespace

bool attn_tc_available() { return encode_fn() != nullptr; }

template <class C>
static int launch_cfg(const AttnParams& p, const specvlm_attn_desc& d, cudaStream_t stream) {
  CUtensorMap mq, mk, mv;
  int rc = make_map(&mq, p.q, d.T, d.H, d.B, d.q_stride_t, d.q_stride_h, d.q_stride_b, tc::kRows);
  if (rc == SPECVLM_OK) rc = make_map(&mk, p.k, d.S_cap, d.H, d.B, d.k_stride_s, d.k_stride_h, d.k_stride_b, C::kTile);
  if (rc == SPECVLM_OK) rc = make_map(&mv, p.v, d.S_cap, d.H, d.B, d.v_stride_s, d.v_stride_h, d.v_stride_b, C::kTile);
  if (rc != SPECVLM_OK) return rc;

  static bool attr_set[64] = {};
  static std::mutex attr_mu;
  std::lock_guard<std::mutex> attr_lock(attr_mu);
  int dev = 0;
  rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice");
  if (rc != SPECVLM_OK) return rc;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    rc = check_cuda(cudaFuncSetAttribute(tree_attn_tc_kernel<C>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         C::kSmemBytes),
                    "attn (tcgen05) smem attribute");
    if (rc != SPECVLM_OK) return rc;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.splits, d.H, d.B);
  cfg.blockDim = dim3(tc::kThreads);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = p.splits;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  // The kernel may be scheduled while the preceding kernel on the stream drains; it orders its own
  // reads and writes with griddepcontrol.wait according to the descriptor flags.
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return check_cuda(cudaLaunchKernelEx(&cfg, tree_attn_tc_kernel<C>, p, mq, mk, mv), "tree_verify_attn (tcgen05) launch");
}

int attn_tc_tile(const specvlm_attn_desc&) { return tc::CfgThroughput::kTile; }

int launch_attn_tc(const AttnParams& p, const specvlm_attn_desc& d, cudaStream_t stream) {
  if (!attn_tc_available()) return fail(SPECVLM_ERR_UNSUPPORTED, "tensor-map encoder not available from the driver");
  // Launches that the caller declares independent of their predecessor run in the half-SM
  // configuration so that consecutive launches overlap; so do launches with more CTAs than SMs,
  // which would otherwise need a second wave. All others get the whole SM.
  const int64_t ctas = static_cast<int64_t>(d.B) * d.H * p.splits;
  if ((d.flags & (SPECVLM_ATTN_FLAG_INPUTS_STABLE | SPECVLM_ATTN_FLAG_HALF_SM)) || ctas > sm_count())
    return launch_cfg<tc::CfgThroughput>(p, d, stream);
  return launch_cfg<tc::CfgLatency>(p, d, stream);
}

}  // namespace specvlm
