/*
 * specvlm.h -- C ABI of the B200 (sm_100a) tree-verification library.
 *
 * The library implements the target model's verification step of EAGLE-2-style
 * speculative decoding for LLaVA-class VLMs, as the SpecVLM paper uses it:
 *   - Section 3.1: the target verifies all drafted tokens in one forward pass and
 *     incorrect tokens are discarded;
 *   - Section 3.3 (a): the target's latest token is the root of the draft token tree;
 *   - Section 4.1: the draft is verified with tree attention (top-k 10, 60 tokens);
 *   - Section 3.2: attention streams the whole (visual-token dominated) KV cache from
 *     HBM on every step -- the cost this library is built around;
 *   - abstract / Section 4.1: decoding is lossless with respect to the target.
 *
 * Conventions
 *   - All pointers are DEVICE pointers owned by the caller unless the parameter name
 *     ends in `_host`. The library allocates no device memory. Scratch memory is a
 *     caller-provided `workspace` sized by the matching *_workspace_bytes() call and
 *     zero-filled ONCE (specvlm_workspace_init) before first use; calls leave it ready
 *     for the next call. Two calls that use the same workspace must not overlap on the
 *     GPU.
 *   - Every call only enqueues work on `stream` (a cudaStream_t passed as void*) and
 *     returns; nothing synchronises.
 *   - Return value: SPECVLM_OK or a negative SPECVLM_ERR_* detected on the host before
 *     anything is launched; specvlm_last_error_string() describes the last error of the
 *     calling thread.
 *   - Device-side data problems (bad prefix length, malformed tree) never trap: the
 *     affected sequence is skipped or clamped and SPECVLM_STATUS_* bits are OR-ed into
 *     the optional `status` word (int32 on the device, may be NULL).
 *   - Tree layout: T <= 64 nodes, node 0 is the root, parent[0] = -1, parent[i] < i.
 *     Node t's K/V row lives in cache slot prefix_len[b] + t.
 *   - Element type of q / k_cache / v_cache / out is bfloat16 (passed as uint16_t bit
 *     patterns). head_dim D must be 128. Base pointers and all strides must be
 *     multiples of 8 elements (16 bytes); D is contiguous.
 */
#ifndef SPECVLM_H_
#define SPECVLM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPECVLM_VERSION 100

#if defined(__GNUC__)
#define SPECVLM_API __attribute__((visibility("default")))
#else
#define SPECVLM_API
#endif

#define SPECVLM_OK 0
#define SPECVLM_ERR_INVALID_ARG (-1)
#define SPECVLM_ERR_UNSUPPORTED (-2)
#define SPECVLM_ERR_CUDA (-3)
#define SPECVLM_ERR_BAD_TREE (-4)

/* bits OR-ed into the device-side status word */
#define SPECVLM_STATUS_BAD_PREFIX 1  /* prefix_len[b] < 0 or prefix_len[b] + T > S_cap */
#define SPECVLM_STATUS_BAD_TREE 2    /* parent[0] != -1 or parent[i] outside [0, i)    */
#define SPECVLM_STATUS_BAD_ACCEPT 4  /* accept_len / accepted_idx out of range         */
#define SPECVLM_STATUS_TIMEOUT 8     /* a bounded on-chip wait gave up                  */

/* specvlm_attn_desc.flags */
/* run the older mma.sync kernels instead of the tcgen05 kernel */
#define SPECVLM_ATTN_FLAG_LEGACY_MMA 1
/* The attention kernel is launched so that it may start while the kernel enqueued before it
 * on the same stream is still draining (programmatic dependent launch). By default it reads
 * nothing until that kernel has completed. The two flags below are promises by the caller
 * that let it start reading earlier:
 * PREFIX_STABLE: prefix_len and the cache slots below prefix_len[b] are not written by that
 *   preceding kernel (true in a decoder layer, where the preceding kernel produces only q and
 *   the tree's own K/V rows): prefix tiles are prefetched early; q, the tree arrays and the
 *   tree slots are read only after the preceding kernel has completed.
 * INPUTS_STABLE: nothing this call reads (q, caches, prefix_len, tree arrays) is written by the
 *   preceding kernel: the whole call may overlap with it (back-to-back attention calls on
 *   independent inputs, as in a benchmark). Its writes to `out` are still issued only after the
 *   preceding kernel has completed. A launch with this flag lets its own successor start at
 *   once, so in a run of consecutive INPUTS_STABLE launches each may overlap all launches of the
 *   run before it and the kernel before the run: the promise must hold against all of those.
 * A launch without INPUTS_STABLE lets its successor start only after its own wait for the
 * preceding kernel is over, so everything earlier on the stream is complete by then. */
#define SPECVLM_ATTN_FLAG_PREFIX_STABLE 2
#define SPECVLM_ATTN_FLAG_INPUTS_STABLE 4
/* Run in the configuration that occupies half an SM per thread block (chosen automatically for
 * INPUTS_STABLE launches): use it for a launch that is followed by launches meant to overlap it. */
#define SPECVLM_ATTN_FLAG_HALF_SM 8

#define SPECVLM_MAX_TREE 64
#define SPECVLM_HEAD_DIM 128

/* Shapes and strides (in ELEMENTS) of one layer's attention call. */
typedef struct specvlm_attn_desc {
  int32_t B;      /* sequences                                   */
  int32_t H;      /* heads (multi-head attention: KV heads == H) */
  int32_t T;      /* tree nodes incl. root, 1..64                */
  int32_t D;      /* head dim, must be 128                       */
  int32_t S_cap;  /* cache capacity in token slots per (b, h)    */
  int32_t num_splits; /* KV splits per (b, h); 0 = library chooses */
  float softmax_scale; /* 0 = 1/sqrt(D)                          */
  int32_t flags;  /* SPECVLM_ATTN_FLAG_* bits, normally 0        */
  int64_t q_stride_b, q_stride_h, q_stride_t; /* q  [B][H][T][D] by default */
  int64_t k_stride_b, k_stride_h, k_stride_s; /* K  [B][H][S_cap][D]        */
  int64_t v_stride_b, v_stride_h, v_stride_s; /* V  [B][H][S_cap][D]        */
  int64_t o_stride_b, o_stride_h, o_stride_t; /* out [B][H][T][D]           */
} specvlm_attn_desc;

/* Shapes and strides (in ELEMENTS) of the multi-layer KV cache for compaction. */
typedef struct specvlm_kv_desc {
  int32_t L, B, H, S_cap, D; /* D must be 128 */
  int32_t reserved;
  int64_t stride_l, stride_b, stride_h, stride_s; /* same for K and V */
} specvlm_kv_desc;

/* Shapes and strides (in ELEMENTS) of the RoPE + append call for one layer. */
typedef struct specvlm_rope_desc {
  int32_t B, H, T, D, S_cap; /* D must be 128 */
  float rope_base;           /* 0 = 10000 */
  int64_t qi_stride_b, qi_stride_h, qi_stride_t; /* q_in   [B][H][T][D] */
  int64_t kn_stride_b, kn_stride_h, kn_stride_t; /* k_new  [B][H][T][D] */
  int64_t vn_stride_b, vn_stride_h, vn_stride_t; /* v_new  [B][H][T][D] */
  int64_t qo_stride_b, qo_stride_h, qo_stride_t; /* q_out  [B][H][T][D] */
  int64_t kc_stride_b, kc_stride_h, kc_stride_s; /* k_cache [B][H][S_cap][D] */
  int64_t vc_stride_b, vc_stride_h, vc_stride_s; /* v_cache [B][H][S_cap][D] */
} specvlm_rope_desc;

SPECVLM_API int specvlm_version(void);
SPECVLM_API const char* specvlm_last_error_string(void);

/* Bytes of scratch specvlm_tree_verify_attn needs for this descriptor (split-KV partial
 * results and arrival counters). Host call. */
SPECVLM_API int specvlm_attn_workspace_bytes(const specvlm_attn_desc* desc_host, size_t* bytes_host);

/* Zero-fill a workspace (once, after allocating it). */
SPECVLM_API int specvlm_workspace_init(void* workspace, size_t bytes, void* stream);

/*
 * Tree metadata (tree attention, Section 4.1; root, Section 3.3 (a)).
 *   tree_parent   int32 [B][T]
 *   prefix_len    int32 [B]
 *   mask_bits     uint64 [B][T] out: bit t of mask_bits[b][i] set iff t is i or an
 *                 ancestor of i
 *   depth         int32 [B][T] out (may be NULL): edges from the root
 *   pos           int32 [B][T] out (may be NULL): prefix_len[b] + depth (position id)
 * A malformed tree sets SPECVLM_STATUS_BAD_TREE and yields self-only masks.
 */
SPECVLM_API int specvlm_tree_build(const int32_t* tree_parent, const int32_t* prefix_len, int B, int T,
                       uint64_t* mask_bits, int32_t* depth, int32_t* pos, int32_t* status,
                       void* stream);

/* Host-side validation of one tree (host pointers): parent[0] = -1, parent[i] in [0, i),
 * T in 1..64, and (if draft_tokens_host != NULL) siblings carry distinct tokens.
 * Returns SPECVLM_OK or SPECVLM_ERR_BAD_TREE. */
SPECVLM_API int specvlm_tree_validate_host(const int32_t* tree_parent_host, const int32_t* draft_tokens_host,
                               int T);

/*
 * Parameter-free visual token compression (Section 3.4: pooling and random pruning of the
 * elastic compressor). x: bf16 [B][N][C] visual tokens, C a multiple of 8, contiguous.
 * specvlm_visual_pool: y[b][m] = mean of x[b][m*ratio .. min((m+1)*ratio, N)), fp32
 *   accumulation; y: bf16 [B][ceil(N/ratio)][C].
 * specvlm_visual_prune: y[b][m] = x[b][keep_idx[b][m]] bit for bit (the random choice of the kept
 *   tokens is the caller's input); y: bf16 [B][M][C]; an index outside [0, N) yields a zero row
 *   and sets SPECVLM_STATUS_BAD_ACCEPT.
 */
SPECVLM_API int specvlm_visual_pool(const uint16_t* x, int B, int N, int C, int ratio, uint16_t* y, void* stream);
SPECVLM_API int specvlm_visual_prune(const uint16_t* x, const int32_t* keep_idx, int B, int N, int C, int M,
                         uint16_t* y, int32_t* status, void* stream);

/*
 * Draft-tree construction, step 1 (Section 4.1: top-k 10 expansion): for each of `rows` logits
 * rows (row r starts at logits + r * row_stride, fp32, V entries) the k <= 16 most probable
 * tokens in order (ties: lower token id first) and their log-probabilities
 * log softmax(logits)[token].
 *   tokens int32 [rows][k] out, logprob fp32 [rows][k] out
 */
SPECVLM_API int specvlm_topk_logprob(const float* logits, int rows, int V, int64_t row_stride, int k,
                         int32_t* tokens, float* logprob, void* stream);

/*
 * Draft-tree construction, step 2 (Section 4.1: 60 tokens in total): rerank of all candidates
 * by cumulative score. Candidate 0 is the root (cand_parent = -1), cand_parent[c] < c.
 * The root and the T-1 best-scoring other candidates are kept (ties: lower candidate index
 * first) and relabelled in (depth, score descending, candidate index) order, so that
 * parent < child.
 *   cand_parent int32 [B][C], cand_score fp32 [B][C] (cumulative log-probability, compared
 *   exactly), cand_token int32 [B][C]; T <= C <= 1024
 *   tree_parent int32 [B][T] out, draft_tokens int32 [B][T] out
 *   kept_candidates int32 [B][T] out (may be NULL): candidate id of every tree node
 *   mask_bits uint64 [B][T], depth int32 [B][T], pos int32 [B][T] out (each may be NULL;
 *   pos = prefix_len[b] + depth needs prefix_len)
 * Scores must not increase from parent to child (log-probabilities are <= 0); otherwise a kept
 * node's parent may be missing and SPECVLM_STATUS_BAD_TREE is set.
 */
SPECVLM_API int specvlm_tree_rerank(const int32_t* cand_parent, const float* cand_score, const int32_t* cand_token,
                        const int32_t* prefix_len, int B, int C, int T, int32_t* tree_parent,
                        int32_t* draft_tokens, int32_t* kept_candidates, uint64_t* mask_bits,
                        int32_t* depth, int32_t* pos, int32_t* status, void* stream);

/*
 * Positioned inputs for tree attention (Section 4.1; the LLaVA targets of Section 4.1 are
 * LLaMA/Vicuna decoders with rotary position embedding). For every sequence b, head h and
 * tree node t, with pos = prefix_len[b] + depth(t):
 *     q_out[b][h][t]                       = RoPE(q_in[b][h][t], pos)
 *     k_cache[b][h][prefix_len[b] + t]     = RoPE(k_new[b][h][t], pos)
 *     v_cache[b][h][prefix_len[b] + t]     = v_new[b][h][t]
 * RoPE rotates the pairs (d, d + 64) by the angle pos * base^(-2d/128). bf16 in and out,
 * angles reduced in double, rotation in fp32. q_out may alias q_in. No other cache byte is
 * written. pos_out (int32 [B][T], may be NULL) receives the position ids. A malformed tree or
 * a prefix that does not fit sets status bits and skips that sequence.
 */
SPECVLM_API int specvlm_rope_append(const uint16_t* q_in, const uint16_t* k_new, const uint16_t* v_new,
                        const int32_t* prefix_len, const int32_t* tree_parent, uint16_t* q_out,
                        uint16_t* k_cache, uint16_t* v_cache, const specvlm_rope_desc* desc_host,
                        int32_t* pos_out, int32_t* status, void* stream);

/*
 * Tree-verification attention for ONE layer (Sections 3.1, 3.2, 4.1).
 * For each sequence b, head h and tree node i < T:
 *     out[b][h][i][:] = softmax_j( q[b][h][i] . K[b][h][j] * scale ) V[b][h][j][:]
 * over keys j < prefix_len[b] (all visible) and j = prefix_len[b] + t, t < T, visible
 * iff bit t of tree_mask_bits[b][i] is set. Slots >= prefix_len[b] + T are never read
 * into the result (they may hold any bit pattern). A node with no visible key gets zeros.
 *   q, out            bf16, strides from desc
 *   k_cache, v_cache  bf16, this layer's cache, strides from desc; read-only here
 *   prefix_len        int32 [B]
 *   tree_parent       int32 [B][T]; used only when tree_mask_bits == NULL (the mask is
 *                     then derived from it); may be NULL otherwise
 *   tree_mask_bits    uint64 [B][T] or NULL
 *   workspace         from specvlm_attn_workspace_bytes, zero-initialised once
 * bf16 inputs, fp32 accumulation, bf16 output.
 */
SPECVLM_API int specvlm_tree_verify_attn(const uint16_t* q, const uint16_t* k_cache, const uint16_t* v_cache,
                             const int32_t* prefix_len, const int32_t* tree_parent,
                             const uint64_t* tree_mask_bits, uint16_t* out,
                             const specvlm_attn_desc* desc_host, void* workspace,
                             int32_t* status, void* stream);

/*
 * Same computation and arguments as specvlm_tree_verify_attn, minus the workspace: the
 * split-KV scratch is a fixed array inside the library (about 16.3 MiB of device memory per
 * GPU, held from the moment the library is loaded on that GPU until the process exits).
 * The paper has no counterpart for this call; it exists for callers that cannot allocate
 * device memory when they need attention: engines whose memory pool already owns all of
 * HBM, decode loops that must avoid the device-wide stall of an allocation, plug-ins that
 * receive raw pointers and no allocator. The call itself allocates nothing and frees
 * nothing.
 *   - Limits: B*H <= 1024 and B*H*splits <= 512, where splits is desc.num_splits or, if
 *     that is 0, the library's choice for the shape. Beyond them the call returns
 *     SPECVLM_ERR_UNSUPPORTED with a message that states the numbers; set desc.num_splits
 *     lower or use the workspace variant.
 *   - The first call on each device looks up the array's device address and raises the
 *     kernel's shared-memory limit; make that first call outside any stream capture, with
 *     the device current.
 *   - All calls on one GPU share the one array. It keeps the previous call's contents; the
 *     call clears the part that must start at zero on `stream` before the kernel runs. Two
 *     calls that overlap on the GPU (different streams, no ordering) race on the array and
 *     give wrong results: order them.
 */
SPECVLM_API int specvlm_tree_verify_attn_static(const uint16_t* q, const uint16_t* k_cache,
                                    const uint16_t* v_cache, const int32_t* prefix_len,
                                    const int32_t* tree_parent, const uint64_t* tree_mask_bits,
                                    uint16_t* out, const specvlm_attn_desc* desc_host,
                                    int32_t* status, void* stream);

/*
 * Greedy target token per tree node (temperature 0; "negligible" sampling cost of
 * Eq. 1): argmax_tokens[b][i] = argmax_v target_logits[b][i][v]; ties -> lowest v;
 * -0 == +0; inputs must be NaN-free.
 *   target_logits  fp32, row r = b*T + i starts at target_logits + r * row_stride
 *                  (row_stride in elements, multiple of 4, >= V)
 *   argmax_tokens  int32 [B][T] out
 */
SPECVLM_API int specvlm_argmax(const float* target_logits, int B, int T, int V, int64_t row_stride,
                   int32_t* argmax_tokens, void* stream);

/*
 * Lossless temperature-0 acceptance (Section 3.1: incorrect tokens are discarded;
 * abstract: lossless). Node i > 0 is kept iff draft_tokens[i] equals the target's greedy
 * token at parent[i] and its parent is kept; the root is always kept. The result is the
 * deepest kept node (lowest index among equals) and its root path.
 *   draft_tokens   int32 [B][T]   (entry 0 = root token, unused by the rule)
 *   tree_parent    int32 [B][T]
 *   target_logits  fp32 [B][T][V] contiguous rows (row stride V), or NULL
 *   argmax_tokens  int32 [B][T]: input when target_logits == NULL; otherwise written
 *                  by an argmax pass first (must be non-NULL in both cases)
 *   accepted_idx   int32 [B][acc_stride] out: node indices of the kept path, entry 0 = 0;
 *                  unused entries = -1; acc_stride >= 1; only the first acc_stride path
 *                  entries are written
 *   accept_len     int32 [B] out: kept DRAFTED tokens (root and bonus token not counted)
 *   next_token     int32 [B] out: the target's greedy token at the last kept node
 */
SPECVLM_API int specvlm_accept(const int32_t* draft_tokens, const int32_t* tree_parent,
                   const float* target_logits, int32_t* argmax_tokens, int B, int T, int V,
                   int32_t* accepted_idx, int acc_stride, int32_t* accept_len,
                   int32_t* next_token, int32_t* status, void* stream);

/*
 * Temperature > 0 acceptance by speculative sampling on the tree (Section 3.1: speculative
 * sampling discards incorrect tokens; Section 4.1: stochastic decoding, target distribution
 * preserved). Children are fixed candidates tried in index order: at the current node with
 * p = softmax(target_logits / temperature), child c with token x is kept iff
 * uniforms_accept[b][c] < p(x) / (1 - mass already rejected at this node); a rejected token is
 * removed from p. If a child is kept the walk descends to it; otherwise next_token is drawn
 * from what is left of p by inverse CDF with uniforms_sample[b][node] (also at a kept leaf).
 *   target_logits    fp32 [B][T][V] contiguous
 *   uniforms_accept  fp32 [B][T] in [0, 1): entry c is used for the keep test of node c
 *   uniforms_sample  fp32 [B][T] in [0, 1): entry u is used if the walk stops at node u
 *   row_stats        fp32 [B][T][2] out, 8-byte aligned: for every node row, max of the logits and
 *                    sum over the vocabulary of exp((logit - max) / temperature); computed by a
 *                    first launch over all rows, read by the walk (so log p(x) of any token at any
 *                    node is (logit - max) / temperature - log(sum))
 *   outputs as in specvlm_accept. fp32 arithmetic; a decision whose random number lies within
 *   rounding distance of its threshold may differ from an exact evaluation.
 */
SPECVLM_API int specvlm_accept_sample(const int32_t* draft_tokens, const int32_t* tree_parent,
                          const float* target_logits, const float* uniforms_accept,
                          const float* uniforms_sample, float temperature, int B, int T, int V,
                          int32_t* accepted_idx, int acc_stride, int32_t* accept_len,
                          int32_t* next_token, float* row_stats, int32_t* status, void* stream);

/*
 * KV compaction after acceptance (the KV cache is the resource the paper's cost model
 * is about, Sections 1 and 3.2). For every layer, for K and V, for every (b, h) and
 * j = 1..accept_len[b]: the 256-byte row in slot prefix_len[b] + accepted_idx[b][j] moves
 * to slot prefix_len[b] + j, in place; all sources of one (layer, b, h) are read before
 * any destination is written. Every other byte of the caches is left untouched.
 * new_prefix_len[b] = prefix_len[b] + 1 + accept_len[b]; it must NOT alias prefix_len.
 */
SPECVLM_API int specvlm_kv_compact(uint16_t* k_cache, uint16_t* v_cache, const specvlm_kv_desc* desc_host,
                       const int32_t* prefix_len, const int32_t* accepted_idx, int acc_stride,
                       const int32_t* accept_len, int32_t* new_prefix_len, int32_t* status,
                       void* stream);

/*
 * Fused path walk + KV gather: specvlm_accept (from argmax_tokens) and specvlm_kv_compact
 * in ONE kernel launch. Every thread block redoes the <= 64-node walk, then moves its share
 * of rows; block 0 also writes accepted_idx / accept_len / next_token / new_prefix_len.
 * Arguments as in the two calls above (argmax_tokens is an input here).
 */
SPECVLM_API int specvlm_accept_compact(const int32_t* draft_tokens, const int32_t* tree_parent,
                           const int32_t* argmax_tokens, int T, uint16_t* k_cache,
                           uint16_t* v_cache, const specvlm_kv_desc* desc_host,
                           const int32_t* prefix_len, int32_t* accepted_idx, int acc_stride,
                           int32_t* accept_len, int32_t* next_token, int32_t* new_prefix_len,
                           int32_t* status, void* stream);

/*
 * The whole verify step of an L-layer decoder in one host call (Sections 3.1, 3.2, 4.1): L
 * attention launches (layer l uses q + l * q_stride_l, the layer-l slice of the caches and
 * out + l * out_stride_l; q and out are [B][H][T][D] contiguous per layer), then
 * specvlm_argmax over target_logits (fp32 [B][T][V] contiguous, V a multiple of 4), then
 * specvlm_accept_compact over all layers. Arguments as in those calls; `workspace` is only
 * needed when the attention call would need one (more than 8 KV splits).
 * layers_independent != 0 declares that no layer's q / cache / out is written by the
 * preceding layer's launch (e.g. precomputed or synthetic per-layer inputs): layers 1..L-1 are
 * then launched with SPECVLM_ATTN_FLAG_INPUTS_STABLE and overlap. In a real decoder, where
 * other kernels sit between the attention calls and feed them, call the per-layer entry points.
 */
SPECVLM_API int specvlm_verify_step(const uint16_t* q, int64_t q_stride_l, uint16_t* k_cache, uint16_t* v_cache,
                        const specvlm_kv_desc* kv_desc_host, const int32_t* prefix_len,
                        const int32_t* tree_parent, const uint64_t* tree_mask_bits,
                        const int32_t* draft_tokens, const float* target_logits, int T, int V,
                        uint16_t* out, int64_t out_stride_l, int32_t* argmax_tokens,
                        int32_t* accepted_idx, int acc_stride, int32_t* accept_len,
                        int32_t* next_token, int32_t* new_prefix_len, int layers_independent,
                        void* workspace, int32_t* status, void* stream);

/*
 * The verify step at temperature > 0 in one host call (Section 4.1 evaluates temperature 1; the
 * target distribution is preserved): the L attention launches as in specvlm_verify_step, then
 * specvlm_accept_sample (speculative sampling along the tree; row statistics, walk and draw), then
 * specvlm_kv_compact over all layers. Arguments as in those calls; acc_stride must cover the
 * deepest path (depth + 1 entries), since the compaction reads accepted_idx.
 */
SPECVLM_API int specvlm_verify_step_sample(const uint16_t* q, int64_t q_stride_l, uint16_t* k_cache,
                        uint16_t* v_cache, const specvlm_kv_desc* kv_desc_host, const int32_t* prefix_len,
                        const int32_t* tree_parent, const uint64_t* tree_mask_bits,
                        const int32_t* draft_tokens, const float* target_logits,
                        const float* uniforms_accept, const float* uniforms_sample, float temperature,
                        int T, int V, uint16_t* out, int64_t out_stride_l, float* row_stats,
                        int32_t* accepted_idx, int acc_stride, int32_t* accept_len, int32_t* next_token,
                        int32_t* new_prefix_len, int layers_independent, void* workspace, int32_t* status,
                        void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SPECVLM_H_ */
