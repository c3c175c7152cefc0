/*
 * snapstream.h -- C ABI of the SnapStream hot path for NVIDIA B200 (sm_100a).
 *
 * SnapStream (arXiv 2511.03092) compresses a prompt's KV cache once, at prefill, into a
 * fixed number of slots  [ sinks | recent-token ring | SnapKV top-K ]  (Section 3.1) and then
 * decodes over that fixed-size cache, writing each new token's K/V into the ring at the index
 * of Eq. 3 (Section 3.3).  This library implements exactly that path:
 *
 *   snap_cache_layout   slot arithmetic of Section 3.1
 *   snap_compress       Section 3.2: Eq. 4 scores -> Eq. 1 window sum -> Eq. 2 pool + top-K ->
 *                       ring construction (Section 3.2.1) and gather into the cache
 *   snap_append_kv      Eq. 3 scatter of one new token per sequence
 *   snap_decode_attn    Section 3.3: (optional Eq. 3 scatter, then) attention of one query token
 *                       per sequence over the valid cache slots
 *
 * and, around it: snap_decode_attn_multi (several new tokens per sequence and step),
 * snap_decode_attn_static (the decode step without a caller-provided scratch buffer),
 * snap_append_kv_concat (the slice-and-concatenate update of Section 3.2.1, as a baseline),
 * snap_prefill_attn + snap_compress_with_row_stats (the prompt's causal attention emitting
 * the normalisers of Eq. 4, and the compression that consumes them),
 * and snap_block_stats + snap_block_select + snap_decode_attn_blocks (a per-step block top-K
 * over the whole middle of the prompt instead of the one-time top-K, the variant the paper's
 * related-work section leaves to future work).
 *
 * Conventions
 *   - "dev" pointers are CUDA device pointers on the current device, "host" pointers are plain
 *     host memory.  Every device buffer must be 16-byte aligned (the tensors, caches, outputs and
 *     workspaces are checked: SNAP_ERR_INVALID_ARG, nothing launched).
 *   - The caller owns every buffer.  The library allocates no device memory; all work is
 *     enqueued on the CUDA stream given and the calls return without synchronising.
 *   - What the library keeps between calls, all of it on the host: per device, the SM count and
 *     which kernels already had their shared-memory limit raised (so the first call of each
 *     entry point on a device must come before any stream capture); per host thread, the
 *     tensor maps of the last few cache buffers the decode kernel was given, keyed on their
 *     addresses and shape; per process, a launch counter and the testing options of
 *     snap_debug_set_option.  Nothing of one call's data outlives the call, except in the fixed
 *     scratch array of snap_decode_attn_static, which says so below.
 *   - Token positions are 0-indexed.  Ls = l_sink, Lr = l_recent, K = topk, Lsr = Ls + Lr,
 *     Sc = Ls + Lr + K, g = n_q_heads / n_kv_heads.
 *   - Element type: all of q, k, v, caches and out share cfg->dtype.
 *   - Return value: SNAP_OK (0) or a negative snap_status.  Nothing throws, aborts or traps.
 *     Conditions only the device can see (a cache slot id out of range, a bounded wait that
 *     ran out, a refinement band that overflowed) are OR-ed into *status_dev when given.
 */
#ifndef SNAPSTREAM_H_
#define SNAPSTREAM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SNAP_F32 0
#define SNAP_BF16 1

#define SNAP_POOL_AVG 0
#define SNAP_POOL_MAX 1

typedef enum snap_status {
  SNAP_OK = 0,
  SNAP_ERR_INVALID_ARG = -1,        /* a value outside the documented domain */
  SNAP_ERR_UNSUPPORTED = -2,        /* valid, but no kernel is built for this shape */
  SNAP_ERR_WORKSPACE_TOO_SMALL = -3,
  SNAP_ERR_NULL_POINTER = -4,
  SNAP_ERR_CUDA = -5,               /* a CUDA runtime call failed; see cudaGetLastError */
  SNAP_ERR_STATIC_SCRATCH_EXCEEDED = -6  /* snap_decode_attn_static: the problem needs more than
                                            SNAP_STATIC_SCRATCH_BYTES of scratch; nothing ran */
} snap_status;

/* bits of *status_dev */
#define SNAP_DEV_BAD_SLOT 1u        /* a slot id was outside [0, max_seqs): that sequence was skipped */
#define SNAP_DEV_WAIT_TIMEOUT 2u    /* a bounded wait on an async copy gave up: results invalid */
#define SNAP_DEV_BAND_OVERFLOW 4u   /* snap_compress: a KV head had more candidates within the re-scoring
                                       band of its top-K threshold than the band buffer holds (512, or
                                       256 for layers with more than 2^18 query elements per KV head);
                                       snap_block_select: more than 256 blocks that single precision
                                       cannot tell from the threshold.  That head keeps its
                                       single-precision order.  The results are valid; exactly tied
                                       scores, which go to the lower position in either precision, are
                                       the usual cause */

#define SNAP_DEV_INDEX_CHECK 8u     /* only from the checked build of the library (compiled with
                                       -DSNAP_DEBUG_BOUNDS): a data-dependent index -- a selected
                                       position, a ring slot, an output rank, a band entry -- fell
                                       outside its array; the access was skipped */

/* One attention layer's shape and SnapStream hyper-parameters (appendix table
 * "SnapStream Hyperparameters": sink, top-K, recent, observation window, pooling kernel). */
typedef struct snap_config {
  int32_t n_q_heads;      /* Hq */
  int32_t n_kv_heads;     /* Hkv, divides Hq */
  int32_t d_qk;           /* key/query row length, multiple of 16 */
  int32_t d_v;            /* value row length, multiple of 16, <= 512 */
  int32_t v_aliases_k;    /* 1: latent attention, V row = first d_v elements of the K row, no V buffers */
  int32_t dtype;          /* SNAP_F32 or SNAP_BF16 */
  int32_t l_sink;         /* Ls >= 0 */
  int32_t l_recent;       /* Lr >= 1 */
  int32_t topk;           /* K  >= 0 */
  int32_t l_obs;          /* Lo, 1 <= Lo <= Lr (every candidate precedes every window query) */
  int32_t pool_kernel;    /* w, odd >= 1 */
  int32_t pool_mode;      /* SNAP_POOL_AVG (Eq. 2) or SNAP_POOL_MAX */
  float softmax_scale;    /* Eq. 4's 1/sqrt(d), supplied by the caller */
  int32_t max_seqs;       /* number of cache slots (sequences resident at once) */
} snap_config_t;

/* Section 3.1: where the three sections live, and the strides of the caches.
 * K cache: [max_seqs][Hkv][Sc][d_qk], V cache: [max_seqs][Hkv][Sc][d_v], row-major, dense. */
typedef struct snap_layout {
  int32_t slots;          /* Sc = Ls + Lr + K  (L_snapstream, Section 3) */
  int32_t sink_off;       /* 0 */
  int32_t ring_off;       /* Ls */
  int32_t topk_off;       /* Ls + Lr */
  int64_t k_row_bytes, v_row_bytes;
  int64_t k_head_stride_bytes, v_head_stride_bytes;   /* Sc * row bytes */
  int64_t k_seq_stride_bytes, v_seq_stride_bytes;     /* Hkv * head stride */
  int64_t k_cache_bytes, v_cache_bytes;               /* max_seqs * seq stride (v: 0 if aliased) */
} snap_layout_t;

/* Section 3.1.  Host only, pure arithmetic.  Validates cfg (INVALID_ARG / UNSUPPORTED). */
int snap_cache_layout(const snap_config_t* cfg, snap_layout_t* out);

/* Bytes of device scratch snap_compress needs for these prompt lengths (cu_seqlens_host has
 * n_seq + 1 entries, prompt i is tokens [cu[i], cu[i+1])).  Negative snap_status on error. */
int64_t snap_compress_workspace_bytes(const snap_config_t* cfg, const int32_t* cu_seqlens_host,
                                      int32_t n_seq);

/* Bytes of device scratch snap_decode_attn needs for n_active sequences. */
int64_t snap_decode_workspace_bytes(const snap_config_t* cfg, int32_t n_active);

/*
 * Prefill compression of n_seq prompts (Section 3.2; appendix listing "SnapStream Prefill KV
 * Cache Compression" describes the same inputs and outputs).
 *
 *   q_obs_dev   [n_seq][Hq][Lo][d_qk]  queries of each prompt's last Lo positions, after any
 *               positional encoding (Section 3.2: encodings are applied before caching).
 *               Ignored (may be NULL) when no prompt has more than Lsr + K tokens.
 *   k_dev,v_dev prompt keys/values, token-major and ragged: element (t, h, c) of prompt i is at
 *               k_dev[(cu[i] + t) * k_token_stride + h * k_head_stride + c]; strides in elements,
 *               multiples of 16 bytes.  v_dev is ignored when cfg->v_aliases_k.
 *   cu_seqlens_host, slot_ids_host   host arrays (n_seq + 1 and n_seq entries); slot_ids give the
 *               cache slot each prompt is compressed into, distinct, in [0, max_seqs).
 *   k_cache_dev, v_cache_dev   the caches (snap_layout_t strides).  For each prompt the whole slot
 *               is rewritten: sinks [0, min(L, Ls)), ring rows of positions [max(Ls, L - Lr), L) at
 *               slot Ls + (p - Ls) mod Lr, selected rows ascending by position from slot Lsr,
 *               zeros elsewhere.
 *   seq_len_dev, valid_topk_dev   [max_seqs] int32; entry slot_ids[i] is set to L_i and to
 *               min(max(L_i - Lsr, 0), K).
 *   topk_idx_dev  NULL, or [n_seq][Hkv][K] int32 receiving the selected absolute positions,
 *               ascending, -1 after the valid ones.
 *   A prompt with L <= Lsr + K is not scored: all its candidates are kept.  Otherwise the K
 *   largest pooled scores win, ties to the lower position.
 *   Precision of the selection: scores are computed in single precision (the part of their error
 *   that can reorder two pooled scores was measured at 1e-7 relative, 2.2e-7 at most, on 32k-
 *   to 128k-token prompts); every candidate whose pooled score lies within 1e-4 relative of the
 *   K-th largest (2e-5 for layers with more than 2^18 query elements per KV head, such as the
 *   latent layout) is then scored again in double precision from q_obs and k, with the
 *   normalisers of Eq. 4 from the single-precision pass, and the order inside that band decides
 *   (measured order error 2e-9, 1.3e-8 at most).  Pooling kernels wider than 33 are not
 *   re-scored.  SNAP_DEV_BAND_OVERFLOW reports a band that did not fit its buffer.
 */
int snap_compress(const snap_config_t* cfg, const snap_layout_t* layout,
                  const void* q_obs_dev,
                  const void* k_dev, int64_t k_token_stride, int64_t k_head_stride,
                  const void* v_dev, int64_t v_token_stride, int64_t v_head_stride,
                  const int32_t* cu_seqlens_host, const int32_t* slot_ids_host, int32_t n_seq,
                  void* k_cache_dev, void* v_cache_dev,
                  int32_t* seq_len_dev, int32_t* valid_topk_dev,
                  int32_t* topk_idx_dev,
                  void* workspace_dev, size_t workspace_bytes,
                  uint32_t* status_dev, void* cuda_stream);

/*
 * Causal attention of n_seq whole prompts that also yields the denominators of Eq. 4
 * (Section 3.2.2 names the score recomputation as the step left to optimise: the normalisers
 * of the observation window's scores are by-products of the prompt's own attention pass).
 *
 *   q_dev     [T][Hq][d_qk] dense, token-major and ragged like k_dev (T = cu[n_seq]); the
 *             queries after positional encoding
 *   k_dev, v_dev and their strides: as in snap_compress
 *   out_dev   [T][Hq][d_v] dense: row t of head h is softmax(scale * q_t . K[0..t]^T) V[0..t]
 *             over the keys of KV head h / (Hq/Hkv) of the same prompt
 *   row_mu_dev  NULL, or [n_seq][Hq][Lo] float: for the prompt's last Lo positions (entry i is
 *             position L - Lo + i; entries of positions below 0 are left untouched)
 *               log2( sum over candidates j in [Ls, L - Lr) of exp(scale * q . k_j) ),
 *             -inf when the prompt has no candidate.  This is what snap_compress_with_row_stats
 *             takes in place of its own first pass over the keys.
 * bf16 layers with d_qk = d_v = 128 and a separate V run on the tensor cores; every other layer
 * (fp32, other head sizes, the latent layout, where v_dev is ignored) runs on a portable kernel
 * that is there for coverage, not for speed.
 * Needs no workspace.  cfg is validated as a whole (as by snap_cache_layout); the kernels use its
 * model-shape fields, l_sink, l_recent, l_obs and softmax_scale.  Errors: SNAP_ERR_NULL_POINTER,
 * SNAP_ERR_INVALID_ARG (cfg, offsets that decrease, strides that are not multiples of 16 bytes):
 * nothing was launched; SNAP_ERR_CUDA: a launch failed.
 */
int snap_prefill_attn(const snap_config_t* cfg, const void* q_dev,
                      const void* k_dev, int64_t k_token_stride, int64_t k_head_stride,
                      const void* v_dev, int64_t v_token_stride, int64_t v_head_stride,
                      const int32_t* cu_seqlens_host, int32_t n_seq,
                      void* out_dev, float* row_mu_dev,
                      uint32_t* status_dev, void* cuda_stream);

/*
 * snap_compress with the Eq. 4 normalisers supplied by the caller (row_mu_dev as written by
 * snap_prefill_attn; NULL = compute them here, which is snap_compress): the score kernel then
 * makes one pass over the candidate keys instead of two.  Same arguments, results, workspace
 * and errors as snap_compress otherwise; every score kernel takes them.  The selection can
 * differ from snap_compress's only where two pooled scores are equal to within single-precision
 * rounding.
 */
int snap_compress_with_row_stats(const snap_config_t* cfg, const snap_layout_t* layout,
                  const void* q_obs_dev, const float* row_mu_dev,
                  const void* k_dev, int64_t k_token_stride, int64_t k_head_stride,
                  const void* v_dev, int64_t v_token_stride, int64_t v_head_stride,
                  const int32_t* cu_seqlens_host, const int32_t* slot_ids_host, int32_t n_seq,
                  void* k_cache_dev, void* v_cache_dev,
                  int32_t* seq_len_dev, int32_t* valid_topk_dev,
                  int32_t* topk_idx_dev,
                  void* workspace_dev, size_t workspace_bytes,
                  uint32_t* status_dev, void* cuda_stream);

/*
 * Eq. 3: for each of n_active sequences write the new token's K/V rows
 * (k_new_dev [n_active][Hkv][d_qk], v_new_dev [n_active][Hkv][d_v], dense) into cache slot
 *   L < Ls ? L : (L - Ls + Lr) mod Lr + Ls,   L = seq_len_dev[slot]  (tokens seen so far),
 * then add one to seq_len_dev[slot].  slot_ids_dev: [n_active] int32 on the device, distinct.
 */
int snap_append_kv(const snap_config_t* cfg, const snap_layout_t* layout,
                   const void* k_new_dev, const void* v_new_dev,
                   const int32_t* slot_ids_dev, int32_t n_active,
                   void* k_cache_dev, void* v_cache_dev, int32_t* seq_len_dev,
                   uint32_t* status_dev, void* cuda_stream);

/*
 * Section 3.3: one decode step.  With k_new_dev != NULL the new token is first written as in
 * snap_append_kv (and seq_len advanced); then out[i][h] = softmax(scale * q[i][h] . K^T) V over
 * the valid slots of sequence i: [0, min(len, Lsr)) and [Lsr, Lsr + valid_topk).
 * With k_new_dev == NULL the cache is only read.
 *   q_dev [n_active][Hq][d_qk], out_dev [n_active][Hq][d_v], dense.  A sequence with no valid
 *   slot gets zeros.  Sequences in one call must use distinct slots.
 */
int snap_decode_attn(const snap_config_t* cfg, const snap_layout_t* layout,
                     const void* q_dev, const void* k_new_dev, const void* v_new_dev,
                     const int32_t* slot_ids_dev, int32_t n_active,
                     void* k_cache_dev, void* v_cache_dev,
                     int32_t* seq_len_dev, const int32_t* valid_topk_dev,
                     void* out_dev,
                     void* workspace_dev, size_t workspace_bytes,
                     uint32_t* status_dev, void* cuda_stream);

/*
 * A decode step with q_len new tokens per sequence (the multi-token prediction that the
 * throughput evaluation of Section 5 assumes: several tokens per forward pass over the same
 * cache).  Defined as q_len steps of
 * snap_decode_attn: token u is appended as in Eq. 3, then query u attends over the cache as it
 * is after tokens 0..u -- a window row that token u evicts is still seen by the queries before
 * u and by none from u on.
 *   q_dev     [n_active][q_len][Hq][d_qk]
 *   k_new_dev [n_active][q_len][Hkv][d_qk], v_new_dev [n_active][q_len][Hkv][d_v]   (required)
 *   out_dev   [n_active][q_len][Hq][d_v];  seq_len_dev[slot] += q_len
 * 1 <= q_len <= Lr (SNAP_ERR_INVALID_ARG otherwise).  bf16 layers with 64-, 128- or 256-wide heads
 * and up to 16 query heads per KV head take 16 / (Hq / Hkv) tokens per pass over the cache (all
 * q_len in one pass when q_len * (Hq / Hkv) <= 16, otherwise several passes, each reading its
 * tokens' rows in place); every other layer (fp32, the latent layout -- v_new_dev is then ignored
 * --) is served as the definition reads, q_len single steps: same results, no saving in cache
 * traffic.  The tcgen05 latent kernel reads each token's rows in place; the other single-step
 * kernels have them staged in the workspace first.
 * Scratch: snap_decode_multi_workspace_bytes(cfg, n_active, q_len).
 */
int64_t snap_decode_multi_workspace_bytes(const snap_config_t* cfg, int32_t n_active, int32_t q_len);
int snap_decode_attn_multi(const snap_config_t* cfg, const snap_layout_t* layout,
                           const void* q_dev, const void* k_new_dev, const void* v_new_dev,
                           const int32_t* slot_ids_dev, int32_t n_active, int32_t q_len,
                           void* k_cache_dev, void* v_cache_dev,
                           int32_t* seq_len_dev, const int32_t* valid_topk_dev,
                           void* out_dev,
                           void* workspace_dev, size_t workspace_bytes,
                           uint32_t* status_dev, void* cuda_stream);

/* Size of the scratch array built into the library for snap_decode_attn_static. */
#define SNAP_STATIC_SCRATCH_BYTES (8u << 20)

/*
 * A decode step for callers that cannot allocate.  (The paper has no counterpart; this is a
 * property of the library, not of the method.)
 *
 * Same operation, arguments and results as snap_decode_attn, but without the workspace
 * arguments: the per-split partial results go to a fixed SNAP_STATIC_SCRATCH_BYTES array that
 * lives inside the library, so the call performs no cudaMalloc/cudaFree and needs no buffer
 * from the caller beyond the inputs and outputs.  It is meant for code that must not allocate
 * where decode steps are issued: a serving loop whose device memory was partitioned up front
 * and is full, a plugin running inside another runtime's callback, a process under a policy
 * that treats late allocations as failures.
 *
 *   - Every GPU that loads this library holds the array from load until process exit.
 *   - The step runs the same kernels with the same split count as snap_decode_attn (the latent
 *     layout included) and needs snap_decode_workspace_bytes(cfg, n_active) - 256 bytes of the
 *     array: n_active * n_q_heads * splits * (d_v + 2) floats (d_v + 4 for the latent layout),
 *     splits being the library's choice for that batch size.  If that exceeds the array the call returns
 *     SNAP_ERR_STATIC_SCRATCH_EXCEEDED and launches nothing; use snap_decode_attn instead.
 *     The 32-sequence, 32-head, d_v = 128 batch of a Llama-3.1-8B layer needs about 4.3 MB.
 *   - All calls share the one array and it keeps the previous call's contents.  Nothing has to
 *     be cleared (every partial that is read was written by the same call), but two calls
 *     that can overlap on the GPU -- different streams without a dependency -- race.
 *   - The first call on each device looks up the array's device address (no allocation);
 *     make that first call outside any stream capture, with that device current.
 */
int snap_decode_attn_static(const snap_config_t* cfg, const snap_layout_t* layout,
                            const void* q_dev, const void* k_new_dev, const void* v_new_dev,
                            const int32_t* slot_ids_dev, int32_t n_active,
                            void* k_cache_dev, void* v_cache_dev,
                            int32_t* seq_len_dev, const int32_t* valid_topk_dev,
                            void* out_dev, uint32_t* status_dev, void* cuda_stream);

/*
 * Section 3.2.1's counter-example, as a measured baseline: the rolling window kept in position
 * order and updated by slicing and concatenating, which yields a NEW cache every step.
 * For each active sequence (L = seq_len_dev[slot]), rows of the output cache are
 *   L <  Ls + Lr:  the input rows, with row L replaced by the new token (a plain scatter);
 *   L >= Ls + Lr:  sinks [0, Ls) and selected rows [Ls+Lr, Sc) copied, window row r takes input
 *                  row r + 1 for Ls <= r < Ls+Lr-1, and the new token goes to row Ls+Lr-1.
 * Then seq_len_dev[slot] += 1.  Slots that are not listed in slot_ids_dev are not copied.
 * The output buffers must differ from the input buffers (SNAP_ERR_INVALID_ARG otherwise); both
 * have the cache layout of snap_cache_layout and are owned by the caller.  A cache that
 * snap_compress built has its window in ring order (Eq. 3); it is in position order as well
 * exactly when (L - Ls) is a multiple of Lr or L <= Ls + Lr.  snap_decode_attn with
 * k_new_dev == NULL reads either order, since attention does not depend on the row order.
 * Traffic per step: the whole cache read and written, against one row for snap_append_kv.
 */
int snap_append_kv_concat(const snap_config_t* cfg, const snap_layout_t* layout,
                          const void* k_new_dev, const void* v_new_dev,
                          const int32_t* slot_ids_dev, int32_t n_active,
                          const void* k_cache_in_dev, const void* v_cache_in_dev,
                          void* k_cache_out_dev, void* v_cache_out_dev,
                          int32_t* seq_len_dev, uint32_t* status_dev, void* cuda_stream);

/*
 * Per-step block top-K (the paper's related-work section: KV blocks with pre-computed statistics,
 * of which the top ones are looked up for every newly decoded token, left there to future
 * work; the criterion is the published query-aware one).  The paper fixes nothing further, so
 * the definition is this library's:
 *   - the cache is built by snap_compress with a top-K budget of at least the prompt's middle
 *     (topk >= L - Ls - Lr): every candidate is then kept, in position order, in the third
 *     section, valid_topk rows of it;
 *   - that section is cut into blocks of block_tokens consecutive rows (a multiple of 16, at
 *     most 1024; the last block may be shorter); a block's statistics are the element-wise
 *     minimum and maximum of its keys per KV head;
 *   - a decode query scores block b of KV head kvh by
 *       U = sum over the query heads h of kvh and the dims d of max(q[h][d] * kmin[b][d], q[h][d] * kmax[b][d]),
 *     an upper bound of the group-summed logit of every key of the block, and the n_blocks
 *     highest-scoring blocks are attended, ties to the lower block index, together with the
 *     sinks and the rolling window, which behave as in snap_decode_attn (Eq. 3 append
 *     included); rows that leave the window during decoding are dropped as before.
 * bf16 layers with 64-, 128- or 256-wide heads, a separate V and at most 16 query heads per KV
 * head; at most 8192 blocks per sequence; SNAP_ERR_UNSUPPORTED otherwise.  The scores are summed
 * in single precision for every block; the blocks that single precision cannot tell from the
 * last selected one (a rigorous error bound per block) are scored again in double precision and
 * ranked by that, so the selection is the one the exact scores give down to relative differences
 * of about 1e-15.  More than 256 such blocks for one (sequence, KV head): the single-precision
 * order stands and SNAP_DEV_BAND_OVERFLOW is raised in *status_dev.
 *
 * snap_block_stats    once per prompt, after snap_compress:
 *   stats_dev  out [max_seqs][Hkv][ceil(topk / block_tokens)][2][d_qk] in the cache's dtype (minimum, then
 *              maximum), snap_block_stats_bytes(cfg, block_tokens) bytes; the blocks of slot_ids_dev[0 .. n_seqs)
 *              are written, rows of blocks past a prompt's last one are left alone.
 * snap_block_select   every step, before the attention:
 *   q_dev [n_active][Hq][d_qk];  block_idx_dev out [n_active][Hkv][n_blocks] ascending block numbers;
 *   n_selected_dev out [n_active][Hkv] = min(n_blocks, blocks of that prompt);
 *   scratch: snap_block_select_workspace_bytes(cfg, n_active, block_tokens) (the scores of every block).
 * snap_decode_attn_blocks   snap_decode_attn that visits only the listed blocks of the third section
 *   (arguments as there, plus the two arrays snap_block_select wrote, same n_blocks);
 *   scratch: snap_decode_blocks_workspace_bytes(cfg, n_active, block_tokens, n_blocks).
 * All three enqueue on cuda_stream and return; device-side conditions go to status_dev.
 */
int64_t snap_block_stats_bytes(const snap_config_t* cfg, int32_t block_tokens);
int snap_block_stats(const snap_config_t* cfg, const snap_layout_t* layout, const int32_t* slot_ids_dev,
                     int32_t n_seqs, const void* k_cache_dev, const int32_t* valid_topk_dev,
                     int32_t block_tokens, void* stats_dev, uint32_t* status_dev, void* cuda_stream);
int snap_block_select(const snap_config_t* cfg, const snap_layout_t* layout, const void* q_dev,
                      const int32_t* slot_ids_dev, int32_t n_active, const void* stats_dev,
                      const int32_t* valid_topk_dev, int32_t block_tokens, int32_t n_blocks,
                      int32_t* block_idx_dev, int32_t* n_selected_dev, void* workspace_dev, size_t workspace_bytes,
                      uint32_t* status_dev, void* cuda_stream);
int64_t snap_block_select_workspace_bytes(const snap_config_t* cfg, int32_t n_active, int32_t block_tokens);
int64_t snap_decode_blocks_workspace_bytes(const snap_config_t* cfg, int32_t n_active, int32_t block_tokens,
                                           int32_t n_blocks);
int snap_decode_attn_blocks(const snap_config_t* cfg, const snap_layout_t* layout, const void* q_dev,
                            const void* k_new_dev, const void* v_new_dev, const int32_t* slot_ids_dev,
                            int32_t n_active, void* k_cache_dev, void* v_cache_dev, int32_t* seq_len_dev,
                            const int32_t* valid_topk_dev, int32_t block_tokens, int32_t n_blocks,
                            const int32_t* block_idx_dev, const int32_t* n_selected_dev, void* out_dev,
                            void* workspace_dev, size_t workspace_bytes, uint32_t* status_dev, void* cuda_stream);

/*
 * Testing and tuning aids (the paper has no counterpart).  Each option is one non-negative
 * integer, process-wide, 0 by default = the library's own choice; changing one while calls are
 * in flight on other threads is not synchronised.  Every kernel choice yields the same results
 * within the tolerances of the tests; the options exist so that the slower kernels and other
 * split counts can be tested and timed.  At the first use of any option each is seeded once
 * from its environment variable (named on the right); the environment is not read again.
 * Returns the option's previous value, or SNAP_ERR_INVALID_ARG.
 */
#define SNAP_OPT_SCORE_KERNEL 0          /* 1: mma.sync score kernel, 2: SIMT, 3: tcgen05 without CTA pairs  SNAP_SCORE_PATH=mma|simt|single */
#define SNAP_OPT_DECODE_GQA_KERNEL 1     /* 1: packed-FP32 GQA decode kernel; the tensor-core kernel 2: always with a merge
                                               launch, 3: with the in-kernel merge of small batches outside stream capture
                                               too (by default only under capture)   SNAP_DECODE_GQA=simt|split|fused */
#define SNAP_OPT_DECODE_LATENT_KERNEL 2  /* 1: mma.sync latent decode kernel        SNAP_DECODE_MLA=mma      */
#define SNAP_OPT_DECODE_NSPLIT 3         /* n: splits per (sequence, KV head)       SNAP_DECODE_NSPLIT=n     */
#define SNAP_OPT_SCORE_NSPLIT 4          /* n: candidate splits of the longest prompt  SNAP_SCORE_NSPLIT=n   */
#define SNAP_OPT_WIDE_STAGES 5           /* n: ring depth of the wide score kernel  SNAP_WIDE_STAGES=n       */
#define SNAP_OPT_PREFILL_KERNEL 6        /* 1: portable prefill attention kernel    SNAP_PREFILL_PATH=simt   */
#define SNAP_OPT_PREFILL_SINGLE_HEADS 7  /* 1: one head per CTA in prefill attention  SNAP_PREFILL_HEADS=1   */
#define SNAP_OPT_REFINE_OFF 8            /* 1: skip the double-precision re-scoring near the top-K
                                               threshold and near the block-selection threshold
                                               (single-precision order)            SNAP_REFINE=0            */
#define SNAP_OPT_COUNT 9
int snap_debug_set_option(int option, int value);

/* Text for a snap_status value (static storage). */
const char* snap_status_string(int status);

/* Number of kernels this library has launched in this process (for benchmarks' bookkeeping). */
int64_t snap_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SNAPSTREAM_H_ */
