// Launch parameters shared by the attention kernels (legacy mma.sync path and tcgen05 path).
#pragma once

#include <stdint.h>

#include "common.cuh"

namespace specvlm {

struct AttnParams {
  const uint16_t* q;
  const uint16_t* k;
  const uint16_t* v;
  uint16_t* out;
  const int32_t* prefix_len;
  const int32_t* parent;
  const uint64_t* mask;
  int32_t* status;
  int32_t* counters;  // [B*H]
  float* part_ml;     // [B*H][splits][64][2]
  float* part_o;      // [B*H][splits][64][128]
  int B, H, T, S_cap, splits;
  int flags;          // specvlm_attn_desc.flags
  float scale_log2;
  int64_t q_sb, q_sh, q_st, k_sb, k_sh, k_ss, v_sb, v_sh, v_ss, o_sb, o_sh, o_st;
};


// tcgen05 / TMA attention path (attn_tc.cu). Handles 1..8 KV splits per (sequence, head); the
// splits of one (sequence, head) form a thread-block cluster. Returns SPECVLM_OK or an error.
int launch_attn_tc(const AttnParams& p, const specvlm_attn_desc& desc, cudaStream_t stream);
// True when the tcgen05 path can take this call (driver entry point for tensor maps found).
bool attn_tc_available();
// Keys per tile the tcgen05 path will use for this descriptor (bounds the useful split count).
int attn_tc_tile(const specvlm_attn_desc& d);

}  // namespace specvlm
