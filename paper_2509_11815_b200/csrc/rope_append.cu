// Rotary position embedding of the tree's queries and new keys at their tree positions, and
// append of the tree's K/V rows to the cache: the step right before tree-verification attention.
//
// The target verifies the whole draft tree in one forward pass with tree attention (Sections
// 3.1, 4.1); its LLaMA/Vicuna-style layers (Section 4.1 names the LLaVA targets) rotate q and k
// by position. A tree node's position is prefix length + depth, so siblings share a position.
// Rotation: pairs (d, d + 64), angle = pos * base^(-2d/128), base 10000 by default.
//
// One block per (tree node, sequence, group of heads). The 64 angles of the node are computed once: the product
// pos * inv_freq and its reduction modulo 2 pi are done in double (positions reach 10^4, where a
// float product would already be off by more than a bf16 step), sine and cosine in float. The
// warps then loop over heads: q row -> rotated q, new k row -> rotated into cache slot P_b + t,
// new v row -> copied into cache slot P_b + t. Rows are 256 bytes; a lane handles two pairs.
#include "common.cuh"

#include <cuda_bf16.h>
#include <math.h>

namespace specvlm {

constexpr int kRopeThreads = 128;

struct RopeParams {
  const uint16_t* q_in; const uint16_t* k_new; const uint16_t* v_new;
  uint16_t* q_out; uint16_t* k_cache; uint16_t* v_cache;
  const int32_t* prefix_len; const int32_t* parent;
  int32_t* pos_out; int32_t* status;
  int B, H, T, S_cap;
  int64_t qi_sb, qi_sh, qi_st, kn_sb, kn_sh, kn_st, vn_sb, vn_sh, vn_st;
  int64_t qo_sb, qo_sh, qo_st, kc_sb, kc_sh, kc_ss, vc_sb, vc_sh, vc_ss;
  double inv_freq[64];
};

__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&t);
}
__device__ __forceinline__ float2 unpack2(uint32_t u) {
  return __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&u));
}

__global__ void __launch_bounds__(kRopeThreads) rope_append_kernel(const RopeParams p) {
  const int t = blockIdx.x, b = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __shared__ float s_cos[64], s_sin[64];
  __shared__ int s_pos;
  grid_dependency_sync();
  const int prefix = p.prefix_len[b];  // every thread: its latency runs beside the parent walk
  if (threadIdx.x == 0) {
    // depth by walking the parent chain (bounded even for a malformed tree)
    const int32_t* par = p.parent + b * p.T;
    int depth = 0, n = t;
    bool bad = false;
    for (int step = 0; step < SPECVLM_MAX_TREE && n > 0; ++step) {
      const int up = par[n];
      if (up < 0 || up >= n) { bad = true; break; }
      n = up;
      ++depth;
    }
    if (t == 0 && par[0] != -1) bad = true;
    const int P = prefix;
    const bool bad_prefix = P < 0 || P + p.T > p.S_cap;
    if (p.status != nullptr) {
      if (bad) atomicOr(p.status, SPECVLM_STATUS_BAD_TREE);
      if (bad_prefix && t == 0) atomicOr(p.status, SPECVLM_STATUS_BAD_PREFIX);
    }
    s_pos = (bad || bad_prefix) ? -1 : P + depth;
    if (p.pos_out != nullptr) p.pos_out[b * p.T + t] = (bad || bad_prefix) ? -1 : P + depth;
  }
  __syncthreads();
  const int pos = s_pos;
  if (pos < 0) return;  // the sequence is skipped: nothing is written for it
  if (threadIdx.x < 64) {
    const double two_pi = 6.283185307179586476925286766559;
    double ang = static_cast<double>(pos) * p.inv_freq[threadIdx.x];
    ang -= two_pi * floor(ang / two_pi);
    float sn, cs;
    sincosf(static_cast<float>(ang), &sn, &cs);
    s_cos[threadIdx.x] = cs;
    s_sin[threadIdx.x] = sn;
  }
  __syncthreads();
  // lane owns pairs d = 2*lane, 2*lane + 1 (elements d and d + 64)
  const float c0 = s_cos[2 * lane], s0 = s_sin[2 * lane], c1 = s_cos[2 * lane + 1], s1 = s_sin[2 * lane + 1];
  const int slot = prefix + t;
  for (int h = blockIdx.z * (kRopeThreads / 32) + warp; h < p.H; h += gridDim.z * (kRopeThreads / 32)) {
    // all six loads of a head's rows are issued before its first store: q_out may alias q_in,
    // which the compiler has to assume and would otherwise serialise three memory round trips
    const uint32_t* qs = reinterpret_cast<const uint32_t*>(p.q_in + b * p.qi_sb + h * p.qi_sh + t * p.qi_st);
    const uint32_t* ks = reinterpret_cast<const uint32_t*>(p.k_new + b * p.kn_sb + h * p.kn_sh + t * p.kn_st);
    const uint32_t* vs = reinterpret_cast<const uint32_t*>(p.v_new + b * p.vn_sb + h * p.vn_sh + t * p.vn_st);
    const uint32_t q_lo = qs[lane], q_hi = qs[lane + 32];
    const uint32_t k_lo = ks[lane], k_hi = ks[lane + 32];
    const uint32_t v_lo = vs[lane], v_hi = vs[lane + 32];
    uint32_t* qd = reinterpret_cast<uint32_t*>(p.q_out + b * p.qo_sb + h * p.qo_sh + t * p.qo_st);
    uint32_t* kd = reinterpret_cast<uint32_t*>(p.k_cache + b * p.kc_sb + h * p.kc_sh + slot * p.kc_ss);
    uint32_t* vd = reinterpret_cast<uint32_t*>(p.v_cache + b * p.vc_sb + h * p.vc_sh + slot * p.vc_ss);
    {
      const float2 lo = unpack2(q_lo), hi = unpack2(q_hi);
      qd[lane] = pack2(lo.x * c0 - hi.x * s0, lo.y * c1 - hi.y * s1);
      qd[lane + 32] = pack2(hi.x * c0 + lo.x * s0, hi.y * c1 + lo.y * s1);
    }
    {
      const float2 lo = unpack2(k_lo), hi = unpack2(k_hi);
      kd[lane] = pack2(lo.x * c0 - hi.x * s0, lo.y * c1 - hi.y * s1);
      kd[lane + 32] = pack2(hi.x * c0 + lo.x * s0, hi.y * c1 + lo.y * s1);
    }
    vd[lane] = v_lo;
    vd[lane + 32] = v_hi;
  }
}

}  // namespace specvlm

using namespace specvlm;

extern "C" int specvlm_rope_append(const uint16_t* q_in, const uint16_t* k_new, const uint16_t* v_new,
                                   const int32_t* prefix_len, const int32_t* tree_parent, uint16_t* q_out,
                                   uint16_t* k_cache, uint16_t* v_cache, const specvlm_rope_desc* d,
                                   int32_t* pos_out, int32_t* status, void* stream) {
  SPECVLM_REQUIRE(d != nullptr, "rope_append: null descriptor");
  SPECVLM_REQUIRE(d->D == SPECVLM_HEAD_DIM, "rope_append: D must be 128");
  SPECVLM_REQUIRE(d->T >= 1 && d->T <= SPECVLM_MAX_TREE, "rope_append: need 1 <= T <= 64");
  SPECVLM_REQUIRE(d->B >= 0 && d->B <= 65535 && d->H >= 1 && d->S_cap >= d->T, "rope_append: bad shape");
  if (d->B == 0) return SPECVLM_OK;
  SPECVLM_REQUIRE(q_in && k_new && v_new && prefix_len && tree_parent && q_out && k_cache && v_cache,
                  "rope_append: null pointer");
  SPECVLM_REQUIRE(aligned16(q_in) && aligned16(k_new) && aligned16(v_new) && aligned16(q_out) &&
                      aligned16(k_cache) && aligned16(v_cache),
                  "rope_append: tensors must be 16-byte aligned");
  SPECVLM_REQUIRE(d->rope_base >= 0.f && isfinite(d->rope_base), "rope_append: bad rope_base");
  const int64_t st[] = {d->qi_stride_b, d->qi_stride_h, d->qi_stride_t, d->kn_stride_b, d->kn_stride_h,
                        d->kn_stride_t, d->vn_stride_b, d->vn_stride_h, d->vn_stride_t, d->qo_stride_b,
                        d->qo_stride_h, d->qo_stride_t, d->kc_stride_b, d->kc_stride_h, d->kc_stride_s,
                        d->vc_stride_b, d->vc_stride_h, d->vc_stride_s};
  for (int64_t s : st) SPECVLM_REQUIRE(s >= 0 && (s % 8) == 0, "rope_append: strides must be non-negative multiples of 8");
  RopeParams p;
  p.q_in = q_in; p.k_new = k_new; p.v_new = v_new; p.q_out = q_out; p.k_cache = k_cache; p.v_cache = v_cache;
  p.prefix_len = prefix_len; p.parent = tree_parent; p.pos_out = pos_out; p.status = status;
  p.B = d->B; p.H = d->H; p.T = d->T; p.S_cap = d->S_cap;
  p.qi_sb = d->qi_stride_b; p.qi_sh = d->qi_stride_h; p.qi_st = d->qi_stride_t;
  p.kn_sb = d->kn_stride_b; p.kn_sh = d->kn_stride_h; p.kn_st = d->kn_stride_t;
  p.vn_sb = d->vn_stride_b; p.vn_sh = d->vn_stride_h; p.vn_st = d->vn_stride_t;
  p.qo_sb = d->qo_stride_b; p.qo_sh = d->qo_stride_h; p.qo_st = d->qo_stride_t;
  p.kc_sb = d->kc_stride_b; p.kc_sh = d->kc_stride_h; p.kc_ss = d->kc_stride_s;
  p.vc_sb = d->vc_stride_b; p.vc_sh = d->vc_stride_h; p.vc_ss = d->vc_stride_s;
  const double base = d->rope_base > 0.f ? static_cast<double>(d->rope_base) : 10000.0;
  for (int i = 0; i < 64; ++i) p.inv_freq[i] = pow(base, -2.0 * i / 128.0);
  // one head per warp (every warp then makes a single memory round trip) while that keeps the grid
  // moderate; larger batches loop over heads inside a warp
  int gz = (d->H + (kRopeThreads / 32) - 1) / (kRopeThreads / 32);
  while (gz > 1 && static_cast<int64_t>(gz) * d->T * d->B > 16384) gz = (gz + 1) / 2;
  dim3 grid(d->T, d->B, gz);
  return check_cuda(launch_overlapped(rope_append_kernel, grid, dim3(kRopeThreads), static_cast<cudaStream_t>(stream), p),
                    "rope_append launch");
}
