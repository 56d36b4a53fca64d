// One call for the whole verify step of a decoder with L layers: L tree-verification attention
// launches (Sections 3.1, 3.2, 4.1), the vocabulary argmax, and the fused acceptance walk + KV
// compaction (Section 3.1: incorrect tokens are discarded). It only chains the library's own
// entry points on the caller's stream, so a caller without CUDA graphs pays one host call per
// step instead of L + 2. specvlm_verify_step_sample is the temperature > 0 form: acceptance by
// speculative sampling (Section 4.1 evaluates temperature 1), then the compaction.
#include "common.cuh"

namespace {

// The L attention launches of a step; checks the arguments that both step entry points share.
int attention_layers(const uint16_t* q, int64_t q_stride_l, uint16_t* k_cache, uint16_t* v_cache,
                     const specvlm_kv_desc* kv, const int32_t* prefix_len, const int32_t* tree_parent,
                     const uint64_t* tree_mask_bits, int T, uint16_t* out, int64_t out_stride_l,
                     int layers_independent, void* workspace, int32_t* status, void* stream) {
  SPECVLM_REQUIRE(kv != nullptr, "verify_step: null kv descriptor");
  SPECVLM_REQUIRE(kv->L >= 1 && kv->D == SPECVLM_HEAD_DIM, "verify_step: need L >= 1 and D = 128");
  SPECVLM_REQUIRE(q && out && k_cache && v_cache, "verify_step: null pointer");
  SPECVLM_REQUIRE(q_stride_l >= 0 && out_stride_l >= 0 && (q_stride_l % 8) == 0 && (out_stride_l % 8) == 0,
                  "verify_step: layer strides must be non-negative multiples of 8");
  specvlm_attn_desc d = {};
  d.B = kv->B; d.H = kv->H; d.T = T; d.D = kv->D; d.S_cap = kv->S_cap;
  d.q_stride_t = d.o_stride_t = kv->D;
  d.q_stride_h = d.o_stride_h = static_cast<int64_t>(T) * kv->D;
  d.q_stride_b = d.o_stride_b = static_cast<int64_t>(kv->H) * T * kv->D;
  d.k_stride_b = d.v_stride_b = kv->stride_b;
  d.k_stride_h = d.v_stride_h = kv->stride_h;
  d.k_stride_s = d.v_stride_s = kv->stride_s;
  for (int l = 0; l < kv->L; ++l) {
    // Layer 0 follows whatever the caller enqueued last; later layers follow this call's own
    // attention launches and may overlap them when the caller declares the layers' inputs independent.
    d.flags = (layers_independent && l > 0) ? SPECVLM_ATTN_FLAG_INPUTS_STABLE
                                            : (layers_independent ? SPECVLM_ATTN_FLAG_HALF_SM : 0);
    int rc = specvlm_tree_verify_attn(q + l * q_stride_l, k_cache + l * kv->stride_l, v_cache + l * kv->stride_l,
                                      prefix_len, tree_parent, tree_mask_bits, out + l * out_stride_l, &d,
                                      workspace, status, stream);
    if (rc != SPECVLM_OK) return rc;
  }
  return SPECVLM_OK;
}

}  // namespace

extern "C" int specvlm_verify_step(const uint16_t* q, int64_t q_stride_l, uint16_t* k_cache, uint16_t* v_cache,
                                   const specvlm_kv_desc* kv, const int32_t* prefix_len,
                                   const int32_t* tree_parent, const uint64_t* tree_mask_bits,
                                   const int32_t* draft_tokens, const float* target_logits, int T, int V,
                                   uint16_t* out, int64_t out_stride_l, int32_t* argmax_tokens,
                                   int32_t* accepted_idx, int acc_stride, int32_t* accept_len,
                                   int32_t* next_token, int32_t* new_prefix_len, int layers_independent,
                                   void* workspace, int32_t* status, void* stream) {
  int rc = attention_layers(q, q_stride_l, k_cache, v_cache, kv, prefix_len, tree_parent, tree_mask_bits, T, out,
                            out_stride_l, layers_independent, workspace, status, stream);
  if (rc != SPECVLM_OK) return rc;
  rc = specvlm_argmax(target_logits, kv->B, T, V, V, argmax_tokens, stream);
  if (rc != SPECVLM_OK) return rc;
  return specvlm_accept_compact(draft_tokens, tree_parent, argmax_tokens, T, k_cache, v_cache, kv, prefix_len,
                                accepted_idx, acc_stride, accept_len, next_token, new_prefix_len, status, stream);
}

extern "C" int specvlm_verify_step_sample(const uint16_t* q, int64_t q_stride_l, uint16_t* k_cache,
                                          uint16_t* v_cache, const specvlm_kv_desc* kv, const int32_t* prefix_len,
                                          const int32_t* tree_parent, const uint64_t* tree_mask_bits,
                                          const int32_t* draft_tokens, const float* target_logits,
                                          const float* uniforms_accept, const float* uniforms_sample,
                                          float temperature, int T, int V, uint16_t* out, int64_t out_stride_l,
                                          float* row_stats, int32_t* accepted_idx, int acc_stride,
                                          int32_t* accept_len, int32_t* next_token, int32_t* new_prefix_len,
                                          int layers_independent, void* workspace, int32_t* status, void* stream) {
  int rc = attention_layers(q, q_stride_l, k_cache, v_cache, kv, prefix_len, tree_parent, tree_mask_bits, T, out,
                            out_stride_l, layers_independent, workspace, status, stream);
  if (rc != SPECVLM_OK) return rc;
  rc = specvlm_accept_sample(draft_tokens, tree_parent, target_logits, uniforms_accept, uniforms_sample, temperature,
                             kv->B, T, V, accepted_idx, acc_stride, accept_len, next_token, row_stats, status, stream);
  if (rc != SPECVLM_OK) return rc;
  return specvlm_kv_compact(k_cache, v_cache, kv, prefix_len, accepted_idx, acc_stride, accept_len, new_prefix_len,
                            status, stream);
}
