// Internal declarations shared by the kernels and the host entry points of libsnapstream.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "snapstream.h"

namespace snap {

// Sequences handled by one group of compress launches; larger batches are chunked on the host.
constexpr int kMaxBatchSeqs = 64;

// Per-launch description of a chunk of prompts, passed to kernels by value.
struct SeqBatch {
  int n;                          // prompts in this chunk
  int tok_off[kMaxBatchSeqs];     // index of each prompt's first token in k/v
  int len[kMaxBatchSeqs];         // L
  int slot[kMaxBatchSeqs];        // cache slot
  int score_idx[kMaxBatchSeqs];   // index among the scored prompts of the chunk, -1 = not scored
  int seq_of_score[kMaxBatchSeqs];// inverse map: scored index -> prompt index in the chunk
  int n_scored;
  int first_seq;                  // index of the chunk's first prompt in the caller's arrays
};

// Shape constants every kernel needs, derived from snap_config_t once on the host.
struct Shape {
  int Hq, Hkv, g, d_qk, d_v, Ls, Lr, K, Lo, w, pool_mode, v_aliases_k, Sc, max_seqs;
  float scale;
};

struct KVSource {
  const void* k;
  const void* v;
  long long k_tok_stride, k_head_stride, v_tok_stride, v_head_stride;   // elements
};

// Double-precision re-scoring of the candidates near the top-K threshold (topk_refine.cu).
// The selection kernel lists every candidate whose single-precision pooled score lies within
// `rel` (relative) of the K-th largest -- the band -- and counts the candidates above the band;
// the refinement kernel recomputes the band members' pooled scores in double and corrects the
// emitted index list where the order inside the band differs.
struct RefineHead {       // one per (scored prompt, KV head); zeroed by the selection kernel
  int n_band;             // band members found (may exceed cap: then nothing is refined)
  int n_sure;             // candidates above the band: selected whatever the band's order
  int done;               // refinement CTAs of this head that have finished
  int changed;            // out: positions that leave the selection (as many enter it)
  float max_dev;          // out: largest |single / double - 1| over the band's pooled scores
  int gather_done;        // gather CTAs of this head that have finished (counted only when changed > 0)
  int pad[2];
};
struct BandEntry { int idx_flag; float p32; };   // candidate index | (selected in single precision) << 31
struct RefineBuffers {
  RefineHead* head;       // [nz]; NULL = no refinement
  BandEntry* band;        // [nz][cap]
  double* part;           // [nz][cap][chunks][w] column sums of Eq. 1 per block of 256 window rows
  double* mu64;           // [nz][R] Eq. 4 normalisers (log2 domain) as the statistics merge computed them
  int* lists;             // [nz][2][cap] candidate indices leaving / entering the selection (first `changed` of each)
  int cap, chunks;
  float rel;
  int stats_natural;      // 1: `stats` holds (m, 1/l) of natural-base exponentials (SIMT path)
};

struct ScoreBuffers {
  float2* part_stats;   // [n_scored*Hkv][nsplit][R]  (running max, sum of exp) per candidate split
  float2* stats;        // [n_scored*Hkv][R]          (row max m_i, 1 / l_i)
  float* C;             // [n_scored*Hkv][c_stride]   Eq. 1 scores summed over the head group
  float* P;             // [n_scored*Hkv][c_stride]   pooled scores
  int c_stride;         // floats per (prompt, kv head) row of C and P
  int nsplit;
  int chunk_tiles;      // 128-wide tcgen05 score kernel: candidate tiles per CTA (split x covers tiles [x c, x c + c))
  const float* ext_mu;  // NULL, or [prompts][Hq][Lo] log2 normalisers of Eq. 4 computed elsewhere
                        // (the prefill attention kernel): pass 1 and the combine step are skipped
  RefineBuffers ref;
};

extern unsigned long long g_launches;
inline void count_launch() { ++g_launches; }

// Current value of a process-wide testing / tuning option (SNAP_OPT_* of snapstream.h).
int option(int which);

// Body of snap_decode_attn with the scratch passed as a plain pointer (api.cu).
int decode_step_with_scratch(const snap_config_t* cfg, const snap_layout_t* layout, const void* q_dev,
                             const void* k_new_dev, const void* v_new_dev, const int32_t* slot_ids_dev,
                             int32_t n_active, void* k_cache_dev, void* v_cache_dev, int32_t* seq_len_dev,
                             const int32_t* valid_topk_dev, void* out_dev, float* scratch, size_t scratch_bytes,
                             size_t slack_bytes, int too_small, uint32_t* status_dev, void* cuda_stream);

// A kernel's dynamic shared-memory limit is a per-device attribute: raise it once on every
// device the library is used on.  `done` is the caller's per-kernel record (static storage).
constexpr int kMaxDevices = 64;
struct SmemLimit { size_t bytes[kMaxDevices]; };
template <typename Kernel>
inline cudaError_t ensure_dyn_smem(Kernel kernel, size_t bytes, SmemLimit& done) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (done.bytes[dev] >= bytes) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess) done.bytes[dev] = bytes;
  return e;
}

// Launch as a programmatic dependent of whatever precedes it in the stream: the grid may become
// resident (and run whatever it has before its griddepcontrol.wait) while the predecessor drains.
// The kernel must execute griddepcontrol.wait before it touches memory a predecessor may write.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = grid;
  lc.blockDim = block;
  lc.dynamicSmemBytes = smem;
  lc.stream = st;
  lc.attrs = attr;
  lc.numAttrs = 1;
  return cudaLaunchKernelEx(&lc, kernel, static_cast<KArgs>(args)...);
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// --- launchers (each enqueues on `st` and returns cudaGetLastError()) ---
cudaError_t launch_score_simt(int dtype, const Shape& s, const SeqBatch& b, const void* q_obs,
                              const KVSource& src, const ScoreBuffers& buf, cudaStream_t st);
// tensor-core version (bf16, 128-wide heads, g*Lo <= 256)
bool score_mma_supported(int dtype, const Shape& s);
int score_mma_nsplit(const Shape& s, int n_scored, int max_le, int sm_count);
cudaError_t launch_score_mma(const Shape& s, const SeqBatch& b, const void* q_obs, const KVSource& src,
                             const ScoreBuffers& buf, cudaStream_t st);
cudaError_t launch_score_combine_log2(const ScoreBuffers& buf, int nz, int R, cudaStream_t st);
// tcgen05 / TMEM / TMA version (bf16, 128-wide heads, g*Lo = 128 or 256)
bool score_umma_supported(int dtype, const Shape& s);
int score_umma_nsplit(const Shape& s, const int* le, int n_scored, int sm_count, int* chunk_tiles);
cudaError_t launch_score_umma(const Shape& s, const SeqBatch& b, const void* q_obs, const KVSource& src,
                              const ScoreBuffers& buf, uint32_t* status, cudaStream_t st);
// tcgen05 version for wide rows / many window rows (d_qk up to 576, g*Lo a multiple of 128)
bool score_umma_wide_supported(int dtype, const Shape& s);
int score_umma_wide_row_blocks(const Shape& s);
int score_umma_wide_nsplit(const Shape& s, int n_scored, int max_le, int sm_count);
cudaError_t launch_score_umma_wide(const Shape& s, const SeqBatch& b, const void* q_obs, const KVSource& src,
                                   const ScoreBuffers& buf, float* cpart, uint32_t* status, cudaStream_t st);
// causal prefill attention on tcgen05 that also emits Eq. 4's normalisers (bf16, 128-wide heads)
bool prefill_attn_supported(int dtype, const Shape& s);
cudaError_t launch_prefill_attn(const Shape& s, const SeqBatch& b, const void* q, const KVSource& src, void* out,
                                float* mu, uint32_t* status, cudaStream_t st);
// portable version (any element type and head sizes, the latent layout included)
cudaError_t launch_prefill_generic(int dtype, const Shape& s, const SeqBatch& b, const void* q, const KVSource& src,
                                   void* out, float* mu, cudaStream_t st);
cudaError_t launch_pool_topk(const Shape& s, const SeqBatch& b, const ScoreBuffers& buf,
                             int* idx_out, uint32_t* status, cudaStream_t st);
// double-precision re-scoring of the near-threshold band (between the selection and the gather, which applies its verdict)
int refine_row_chunks(const Shape& s);
cudaError_t launch_topk_refine(int dtype, const Shape& s, const SeqBatch& b, const void* q_obs, const KVSource& src,
                               const ScoreBuffers& buf, uint32_t* status, int sm_count, cudaStream_t st);
// `buf` non-NULL with buf->ref.head set: the refinement kernel was launched just before this one
cudaError_t launch_gather(int dtype, const Shape& s, const SeqBatch& b, const KVSource& src,
                          int* idx, void* k_cache, void* v_cache, int* seq_len,
                          int* valid_topk, uint32_t* status, cudaStream_t st, const ScoreBuffers* buf = nullptr);
cudaError_t launch_append(int dtype, const Shape& s, const void* k_new, const void* v_new,
                          const int* slot_ids, int n_active, void* k_cache, void* v_cache,
                          int* seq_len, uint32_t* status, cudaStream_t st);
cudaError_t launch_decode_generic(int dtype, const Shape& s, const void* q, const void* k_new,
                                  const void* v_new, const int* slot_ids, int n_active,
                                  void* k_cache, void* v_cache, int* seq_len,
                                  const int* valid_topk, void* out, float* partials, int nsplit,
                                  uint32_t* status, cudaStream_t st);
int decode_generic_nsplit(const Shape& s, int n_active, int sm_count);
size_t decode_partial_floats(const Shape& s, int n_active, int nsplit);
// grouped-query bf16, 128-wide heads: bulk-async staged streaming kernel
bool decode_gqa_supported(int dtype, const Shape& s);
int decode_gqa_nsplit(const Shape& s, int n_active, int sm_count);
size_t decode_gqa_partial_floats(const Shape& s, int n_active, int nsplit);
cudaError_t launch_decode_gqa(const Shape& s, const void* q, const void* k_new, const void* v_new,
                              const int* slot_ids, int n_active, void* k_cache, void* v_cache,
                              int* seq_len, const int* valid_topk, void* out, float* partials,
                              int nsplit, uint32_t* status, cudaStream_t st);

cudaError_t launch_decode_gqa_merge(const float* partials, void* out, int Hq, int nsplit, const int* slot_ids,
                                    int n_rows, int q_len, int* seq_len, int max_seqs, int bump, cudaStream_t st,
                                    int q_total = 0, int u0 = 0);
// the same on tensor cores (mma.sync, the group's heads on the N side; head sizes 64, 128, 256): cost independent of the group size
bool decode_gqa_mma_supported(int dtype, const Shape& s);
bool decode_use_gqa_mma(int dtype, const Shape& s);     // the choice between the two, shared by all entry points
int decode_gqa_mma_nsplit(const Shape& s, int n_active, int sm_count);
size_t decode_gqa_mma_partial_floats(const Shape& s, int n_rows, int nsplit);
cudaError_t launch_decode_gqa_mma(const Shape& s, const void* q, const void* k_new, const void* v_new,
                                  const int* slot_ids, int n_active, void* k_cache, void* v_cache,
                                  int* seq_len, const int* valid_topk, void* out, float* partials,
                                  int nsplit, uint32_t* status, cudaStream_t st, int q_len = 1, int q_total = 0, int u0 = 0,
                                  const int* block_idx = nullptr, const int* n_sel = nullptr, int blocks_cap = 0,
                                  int block_tokens = 0);
// (q_len tokens per sequence in one pass, q_len * g <= 16: tokens u0 .. u0 + q_len - 1 of the q_total per sequence that
// q, k_new, v_new and out hold; q_total = 0: they hold exactly these)

// (block_idx: per-step block lookup -- only the listed blocks of block_tokens rows of the third section are visited)
// per-step block top-K: statistics of the third section's blocks, and the per-step selection (block_topk.cu)
int block_count_max(const Shape& s, int block_tokens);
bool block_topk_supported(int dtype, const Shape& s, int block_tokens);
cudaError_t launch_block_stats(const Shape& s, int block_tokens, const int* slot_ids, int n, const void* k_cache,
                               const int* valid_topk, void* stats, uint32_t* status, cudaStream_t st);
cudaError_t launch_block_select(const Shape& s, int block_tokens, int n_blocks, const void* q, const int* slot_ids,
                                int n_active, const void* stats, const int* valid_topk, int* block_idx, int* n_sel,
                                void* scratch, uint32_t* status, cudaStream_t st);
size_t block_select_scratch_bytes(const Shape& s, int block_tokens, int n_active);

// latent attention (one 576-wide KV row shared by all heads, V = its first 512 dims): mma.sync kernel
bool decode_mla_supported(int dtype, const Shape& s);
int decode_mla_nsplit(const Shape& s, int n_active, int sm_count);
size_t decode_mla_partial_floats(const Shape& s, int n_active, int nsplit);
cudaError_t launch_decode_mla(const Shape& s, const void* q, const void* k_new, const int* slot_ids,
                              int n_active, void* k_cache, int* seq_len, const int* valid_topk, void* out,
                              float* partials, int nsplit, uint32_t* status, cudaStream_t st);

cudaError_t launch_decode_mla_merge(const float* partials, void* out, int n_active, int Hq, int nsplit,
                                    const int* slot_ids, int* seq_len, int max_seqs, int bump, cudaStream_t st,
                                    bool programmatic = false, int q_len = 1, int u = 0);
// latent attention on tcgen05, streamed: queries in shared memory, cache rows streamed as key slabs and value chunks
bool decode_mla_stream_supported(int dtype, const Shape& s);
int decode_mla_stream_nsplit(const Shape& s, int n_active, int sm_count);
size_t decode_mla_stream_partial_floats(const Shape& s, int n_active, int nsplit);
// q_len > 1: q, k_new and out hold q_len tokens per sequence ([n][q_len][...]) and this call serves token u of each
cudaError_t launch_decode_mla_stream(const Shape& s, const void* q, const void* k_new, const int* slot_ids,
                                     int n_active, void* k_cache, int* seq_len, const int* valid_topk, void* out,
                                     float* partials, int nsplit, uint32_t* status, cudaStream_t st, int q_len = 1, int u = 0);

// Checked indexing for the debugging build (-DSNAP_DEBUG_BOUNDS): a data-dependent index that falls
// outside [0, n) raises SNAP_DEV_INDEX_CHECK in the status word and the access is skipped -- nothing
// traps.  In the regular build the check compiles to `true`.
#ifdef SNAP_DEBUG_BOUNDS
__device__ __forceinline__ bool index_ok(long long i, long long n, uint32_t* status) {
  if (i >= 0 && i < n) return true;
  if (status) atomicOr(status, SNAP_DEV_INDEX_CHECK);
  return false;
}
#else
__device__ __forceinline__ bool index_ok(long long, long long, uint32_t*) { return true; }
#endif

// --- small device helpers ---
template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) {
  return __bfloat162float(x);
}
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) {
  return __float2bfloat16_rn(x);
}

// Eq. 3: cache slot written by the token at 0-indexed position t.
__host__ __device__ __forceinline__ int ring_slot(int t, int Ls, int Lr) {
  return t < Ls ? t : (t - Ls + Lr) % Lr + Ls;
}

}  // namespace snap
