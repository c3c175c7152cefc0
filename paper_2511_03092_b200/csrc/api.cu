// Host side of the C ABI: argument validation, slot arithmetic, scratch planning and the
// launch sequences.  No allocation, no synchronisation.  State kept between calls: the launch
// counter, a per-device SM count, and the process-wide testing options below.
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>

#include "snap_internal.cuh"

namespace snap {

unsigned long long g_launches = 0;

// Testing and tuning options: one integer each, process-wide, set through snap_debug_set_option.
// Each starts from its environment variable, which is read once, at the first use of any option.
namespace {
int g_opt[SNAP_OPT_COUNT] = {};
std::once_flag g_opt_once;

void seed_options() {
  auto env_int = [](const char* name) { const char* e = getenv(name); const int v = e ? atoi(e) : 0; return v > 0 ? v : 0; };
  if (const char* e = getenv("SNAP_SCORE_PATH")) g_opt[SNAP_OPT_SCORE_KERNEL] = !strcmp(e, "mma") ? 1 : !strcmp(e, "simt") ? 2 : !strcmp(e, "single") ? 3 : 0;
  if (const char* e = getenv("SNAP_DECODE_GQA")) g_opt[SNAP_OPT_DECODE_GQA_KERNEL] = !strcmp(e, "simt") ? 1 : !strcmp(e, "split") ? 2 : !strcmp(e, "fused") ? 3 : 0;
  if (const char* e = getenv("SNAP_DECODE_MLA")) g_opt[SNAP_OPT_DECODE_LATENT_KERNEL] = e[0] == 'm';
  if (const char* e = getenv("SNAP_PREFILL_PATH")) g_opt[SNAP_OPT_PREFILL_KERNEL] = !strcmp(e, "simt");
  if (const char* e = getenv("SNAP_PREFILL_HEADS")) g_opt[SNAP_OPT_PREFILL_SINGLE_HEADS] = e[0] == '1';
  if (const char* e = getenv("SNAP_REFINE")) g_opt[SNAP_OPT_REFINE_OFF] = e[0] == '0';
  g_opt[SNAP_OPT_DECODE_NSPLIT] = env_int("SNAP_DECODE_NSPLIT");
  g_opt[SNAP_OPT_SCORE_NSPLIT] = env_int("SNAP_SCORE_NSPLIT");
  g_opt[SNAP_OPT_WIDE_STAGES] = env_int("SNAP_WIDE_STAGES");
}
}  // namespace

int option(int which) {
  std::call_once(g_opt_once, seed_options);
  return which >= 0 && which < SNAP_OPT_COUNT ? g_opt[which] : 0;
}

// 128-wide bf16 heads decode on the tensor-core kernel (faster than the packed-FP32 kernel at every
// group size); option SNAP_OPT_DECODE_GQA_KERNEL = 1 keeps the packed-FP32 kernel (testing aid).
bool decode_use_gqa_mma(int dtype, const Shape& s) {
  if (option(SNAP_OPT_DECODE_GQA_KERNEL) == 1) return false;
  return decode_gqa_mma_supported(dtype, s);
}

namespace {

int sm_count() {
  static int cached[kMaxDevices] = {};
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < kMaxDevices) {
    if (cached[dev] > 0) return cached[dev];
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) {
      cached[dev] = n;
      return n;
    }
  }
  (void)cudaGetLastError();
  return 148;   // B200; used only for sizing when no device is visible
}

int elt_bytes(int dtype) { return dtype == SNAP_F32 ? 4 : 2; }

int validate(const snap_config_t* c) {
  if (!c) return SNAP_ERR_NULL_POINTER;
  if (c->dtype != SNAP_F32 && c->dtype != SNAP_BF16) return SNAP_ERR_INVALID_ARG;
  if (c->n_q_heads < 1 || c->n_kv_heads < 1 || c->n_q_heads % c->n_kv_heads) return SNAP_ERR_INVALID_ARG;
  if (c->d_qk < 16 || c->d_v < 16) return SNAP_ERR_INVALID_ARG;
  if (c->l_sink < 0 || c->l_recent < 1 || c->topk < 0) return SNAP_ERR_INVALID_ARG;
  if (c->l_obs < 1 || c->l_obs > c->l_recent) return SNAP_ERR_INVALID_ARG;
  if (c->pool_kernel < 1 || c->pool_kernel % 2 == 0) return SNAP_ERR_INVALID_ARG;
  if (c->pool_mode != SNAP_POOL_AVG && c->pool_mode != SNAP_POOL_MAX) return SNAP_ERR_INVALID_ARG;
  if (!(c->softmax_scale > 0.f) || !std::isfinite(c->softmax_scale)) return SNAP_ERR_INVALID_ARG;
  if (c->max_seqs < 1) return SNAP_ERR_INVALID_ARG;
  if (c->v_aliases_k != 0 && c->v_aliases_k != 1) return SNAP_ERR_INVALID_ARG;
  if (c->v_aliases_k && c->d_v > c->d_qk) return SNAP_ERR_INVALID_ARG;
  if ((long long)c->l_sink + c->l_recent + c->topk > (1LL << 30)) return SNAP_ERR_INVALID_ARG;
  if (c->d_qk % 16 || c->d_v % 16 || c->d_v > 512 || c->d_qk > 1024) return SNAP_ERR_UNSUPPORTED;
  return SNAP_OK;
}

Shape make_shape(const snap_config_t* c) {
  Shape s;
  s.Hq = c->n_q_heads; s.Hkv = c->n_kv_heads; s.g = s.Hq / s.Hkv; s.d_qk = c->d_qk; s.d_v = c->d_v;
  s.Ls = c->l_sink; s.Lr = c->l_recent; s.K = c->topk; s.Lo = c->l_obs; s.w = c->pool_kernel;
  s.pool_mode = c->pool_mode; s.v_aliases_k = c->v_aliases_k; s.Sc = s.Ls + s.Lr + s.K;
  s.max_seqs = c->max_seqs; s.scale = c->softmax_scale;
  return s;
}

size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }
// Every device buffer must start on a 16-byte boundary (the kernels use 16-byte accesses and bulk copies); a
// pointer that does not is refused here rather than left to fault on the device.  NULL passes: optional
// arguments are checked for presence separately.
template <typename... P>
bool misaligned(const P*... p) { return (((reinterpret_cast<uintptr_t>(p) & 15u) != 0) || ...); }

// Option SNAP_OPT_SCORE_KERNEL = 1 (mma.sync) or 2 (SIMT) forces a slower score kernel, 3 keeps the
// tcgen05 kernels but without CTA pairs (testing aids); default: the best one.
bool forced_legacy_score() { return option(SNAP_OPT_SCORE_KERNEL) == 1 || option(SNAP_OPT_SCORE_KERNEL) == 2; }
bool use_umma(int dtype, const Shape& s) {
  if (forced_legacy_score()) return false;
  return score_umma_supported(dtype, s);
}
bool use_umma_wide(int dtype, const Shape& s) {
  if (forced_legacy_score()) return false;
  return !score_umma_supported(dtype, s) && score_umma_wide_supported(dtype, s);
}
bool use_mma(int dtype, const Shape& s) {
  if (option(SNAP_OPT_SCORE_KERNEL) == 2) return false;
  return score_mma_supported(dtype, s);
}

// Scratch regions of one chunk of prompts (offsets relative to the chunk area).
struct ChunkPlan {
  int n_scored, max_le, nsplit, chunk_tiles, c_stride;
  size_t part_off, stats_off, c_off, p_off, cpart_off, bytes;
  // double-precision refinement of the selection near the threshold (cap == 0: none)
  int ref_cap, ref_chunks;
  float ref_rel;
  size_t ref_band_off, ref_part_off, ref_mu_off, ref_lists_off, ref_head_off;
};

// Band of the refinement: wide (1e-4 relative, up to 512 members) where re-scoring a member is cheap,
// narrower (2e-5, up to 256 members) where one member costs millions of multiply-adds (the latent
// shape: 4096 window rows x 576 dims).  Both are far above the single-precision error of a pooled
// score (measured: 2e-8 .. 6e-7 relative on the benchmark shapes).  Pooling kernels wider than 33
// are not refined.
void plan_refine(const Shape& s, ChunkPlan& p) {
  p.ref_cap = 0;
  if (option(SNAP_OPT_REFINE_OFF) == 1 || s.w > 33 || p.n_scored == 0) return;
  const long long member_cost = (long long)s.g * s.Lo * s.d_qk;
  p.ref_cap = member_cost <= (1LL << 18) ? 512 : 256;
  p.ref_rel = member_cost <= (1LL << 18) ? 1e-4f : 2e-5f;
  p.ref_chunks = refine_row_chunks(s);
}

ChunkPlan plan_chunk(int dtype, const Shape& s, const int32_t* cu, int first, int n) {
  ChunkPlan p;
  std::memset(&p, 0, sizeof(p));
  int le[kMaxBatchSeqs];                                        // candidates of each scored prompt
  for (int i = 0; i < n; ++i) {
    const int L = cu[first + i + 1] - cu[first + i];
    const int Le = L - s.Ls - s.Lr;
    if (s.K > 0 && Le > s.K) {
      le[p.n_scored++] = Le;
      p.max_le = Le > p.max_le ? Le : p.max_le;
    }
  }
  if (p.n_scored == 0) return p;
  const int R = s.g * s.Lo;
  const int row_blocks = (R + 63) / 64;
  const int tiles = (p.max_le + 63) / 64;
  long long nsplit = (2LL * sm_count() + (long long)p.n_scored * s.Hkv * row_blocks - 1) /
                     ((long long)p.n_scored * s.Hkv * row_blocks);
  if (nsplit > tiles) nsplit = tiles;
  if (nsplit > 64) nsplit = 64;
  if (nsplit < 1) nsplit = 1;
  if (use_umma(dtype, s)) p.nsplit = score_umma_nsplit(s, le, p.n_scored, sm_count(), &p.chunk_tiles);
  else if (use_umma_wide(dtype, s)) p.nsplit = score_umma_wide_nsplit(s, p.n_scored, p.max_le, sm_count());
  else if (use_mma(dtype, s)) p.nsplit = score_mma_nsplit(s, p.n_scored, p.max_le, sm_count());
  else p.nsplit = (int)nsplit;
  p.c_stride = (int)align_up((size_t)p.max_le, 64);
  const size_t nz = (size_t)p.n_scored * s.Hkv;
  size_t off = 0;
  p.part_off = off;  off += align_up(nz * p.nsplit * R * sizeof(float2));
  p.stats_off = off; off += align_up(nz * R * sizeof(float2));
  p.c_off = off;     off += align_up(nz * p.c_stride * sizeof(float));
  p.p_off = off;     off += align_up(nz * p.c_stride * sizeof(float));
  p.cpart_off = off;
  if (use_umma_wide(dtype, s)) off += align_up(nz * score_umma_wide_row_blocks(s) * p.c_stride * sizeof(float));
  plan_refine(s, p);
  if (p.ref_cap > 0) {
    p.ref_band_off = off; off += align_up(nz * p.ref_cap * sizeof(BandEntry));
    p.ref_part_off = off; off += align_up(nz * p.ref_cap * p.ref_chunks * s.w * sizeof(double));
    p.ref_mu_off = off;   off += align_up(nz * R * sizeof(double));
    p.ref_lists_off = off; off += align_up(nz * 2 * p.ref_cap * sizeof(int));
    p.ref_head_off = off; off += align_up(nz * sizeof(RefineHead));
  }
  p.bytes = off;
  return p;
}

int check_cu(const int32_t* cu, int n_seq) {
  if (!cu) return SNAP_ERR_NULL_POINTER;
  if (n_seq < 0) return SNAP_ERR_INVALID_ARG;
  for (int i = 0; i < n_seq; ++i)
    if (cu[i + 1] < cu[i]) return SNAP_ERR_INVALID_ARG;
  return SNAP_OK;
}

struct DecodePlan { bool gqa, gqa_mma, mla, mla_stream; int nsplit; size_t floats; };

bool use_gqa_mma(int dtype, const Shape& s) { return decode_use_gqa_mma(dtype, s); }

// Kernel for the latent layout: the streamed tcgen05 kernel when the head count allows (multiples
// of 128), else the mma.sync kernel; option SNAP_OPT_DECODE_LATENT_KERNEL = 1 forces the latter.
bool use_mla_stream(int dtype, const Shape& s) {
  if (option(SNAP_OPT_DECODE_LATENT_KERNEL) == 1) return false;
  return decode_mla_stream_supported(dtype, s);
}

DecodePlan plan_decode(int dtype, const Shape& s, int n_active) {
  DecodePlan p;
  const int n = n_active > 0 ? n_active : 1;
  p.gqa_mma = use_gqa_mma(dtype, s);
  p.gqa = p.gqa_mma || decode_gqa_supported(dtype, s);
  p.mla_stream = !p.gqa && use_mla_stream(dtype, s);
  p.mla = !p.gqa && !p.mla_stream && decode_mla_supported(dtype, s);
  if (p.mla_stream) {
    p.nsplit = decode_mla_stream_nsplit(s, n, sm_count());
    p.floats = decode_mla_stream_partial_floats(s, n_active, p.nsplit);
  } else if (p.mla) {
    p.nsplit = decode_mla_nsplit(s, n, sm_count());
    p.floats = decode_mla_partial_floats(s, n_active, p.nsplit);
  } else if (p.gqa_mma) {
    p.nsplit = decode_gqa_mma_nsplit(s, n, sm_count());
    p.floats = decode_gqa_mma_partial_floats(s, n_active, p.nsplit);
  } else if (p.gqa) {
    p.nsplit = decode_gqa_nsplit(s, n, sm_count());
    p.floats = decode_gqa_partial_floats(s, n_active, p.nsplit);
  } else {
    p.nsplit = decode_generic_nsplit(s, n, sm_count());
    p.floats = decode_partial_floats(s, n_active, p.nsplit);
  }
  return p;
}

size_t idx_bytes(const Shape& s, int n_seq) {
  return align_up((size_t)n_seq * s.Hkv * (s.K > 0 ? s.K : 1) * sizeof(int));
}

}  // namespace

// One decode step with its partial results in `scratch`: the body of snap_decode_attn, shared with
// snap_decode_attn_static so that both choose the same kernel and split count.  `slack_bytes` is
// the margin the size query adds for the caller's own alignment; `too_small` is the status
// returned when the partial results do not fit.
int decode_step_with_scratch(const snap_config_t* cfg, const snap_layout_t* layout, const void* q_dev,
                             const void* k_new_dev, const void* v_new_dev, const int32_t* slot_ids_dev,
                             int32_t n_active, void* k_cache_dev, void* v_cache_dev, int32_t* seq_len_dev,
                             const int32_t* valid_topk_dev, void* out_dev, float* scratch, size_t scratch_bytes,
                             size_t slack_bytes, int too_small, uint32_t* status_dev, void* cuda_stream) {
  const int rc = validate(cfg);
  if (rc != SNAP_OK) return rc;
  if (!layout) return SNAP_ERR_NULL_POINTER;
  if (n_active < 0) return SNAP_ERR_INVALID_ARG;
  if (n_active == 0) return SNAP_OK;
  if (!q_dev || !slot_ids_dev || !k_cache_dev || !seq_len_dev || !valid_topk_dev || !out_dev || !scratch)
    return SNAP_ERR_NULL_POINTER;
  if (!cfg->v_aliases_k && !v_cache_dev) return SNAP_ERR_NULL_POINTER;
  if (k_new_dev && !cfg->v_aliases_k && !v_new_dev) return SNAP_ERR_NULL_POINTER;
  if (misaligned(q_dev, k_new_dev, v_new_dev, k_cache_dev, v_cache_dev, out_dev) || misaligned(scratch)) return SNAP_ERR_INVALID_ARG;
  const Shape s = make_shape(cfg);
  if (layout->slots != s.Sc) return SNAP_ERR_INVALID_ARG;
  const DecodePlan p = plan_decode(cfg->dtype, s, n_active);
  if (scratch_bytes < p.floats * sizeof(float) + slack_bytes) return too_small;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e;
  if (p.mla_stream)
    e = launch_decode_mla_stream(s, q_dev, k_new_dev, slot_ids_dev, n_active, k_cache_dev, seq_len_dev,
                                 valid_topk_dev, out_dev, scratch, p.nsplit, status_dev, st);
  else if (p.mla)
    e = launch_decode_mla(s, q_dev, k_new_dev, slot_ids_dev, n_active, k_cache_dev, seq_len_dev,
                          valid_topk_dev, out_dev, scratch, p.nsplit, status_dev, st);
  else if (p.gqa && p.gqa_mma)
    e = launch_decode_gqa_mma(s, q_dev, k_new_dev, v_new_dev, slot_ids_dev, n_active, k_cache_dev,
                              v_cache_dev, seq_len_dev, valid_topk_dev, out_dev, scratch, p.nsplit, status_dev, st);
  else if (p.gqa)
    e = launch_decode_gqa(s, q_dev, k_new_dev, v_new_dev, slot_ids_dev, n_active, k_cache_dev,
                          v_cache_dev, seq_len_dev, valid_topk_dev, out_dev, scratch, p.nsplit, status_dev, st);
  else
    e = launch_decode_generic(cfg->dtype, s, q_dev, k_new_dev, v_new_dev, slot_ids_dev, n_active,
                              k_cache_dev, v_cache_dev, seq_len_dev, valid_topk_dev, out_dev, scratch, p.nsplit,
                              status_dev, st);
  return e == cudaSuccess ? SNAP_OK : SNAP_ERR_CUDA;
}

}  // namespace snap

using namespace snap;

extern "C" {

const char* snap_status_string(int status) {
  switch (status) {
    case SNAP_OK: return "ok";
    case SNAP_ERR_INVALID_ARG: return "invalid argument";
    case SNAP_ERR_UNSUPPORTED: return "unsupported shape";
    case SNAP_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case SNAP_ERR_NULL_POINTER: return "null pointer";
    case SNAP_ERR_CUDA: return "CUDA error";
    case SNAP_ERR_STATIC_SCRATCH_EXCEEDED: return "problem exceeds the built-in static scratch";
    default: return "unknown status";
  }
}

int64_t snap_kernel_launch_count(void) { return (int64_t)g_launches; }

int snap_debug_set_option(int opt, int value) {
  if (opt < 0 || opt >= SNAP_OPT_COUNT || value < 0) return SNAP_ERR_INVALID_ARG;
  const int old = option(opt);
  g_opt[opt] = value;
  return old;
}

int snap_cache_layout(const snap_config_t* cfg, snap_layout_t* out) {
  if (!cfg || !out) return SNAP_ERR_NULL_POINTER;
  const int rc = validate(cfg);
  if (rc != SNAP_OK) return rc;
  const int eb = elt_bytes(cfg->dtype);
  out->slots = cfg->l_sink + cfg->l_recent + cfg->topk;
  out->sink_off = 0;
  out->ring_off = cfg->l_sink;
  out->topk_off = cfg->l_sink + cfg->l_recent;
  out->k_row_bytes = (int64_t)cfg->d_qk * eb;
  out->v_row_bytes = (int64_t)cfg->d_v * eb;
  out->k_head_stride_bytes = out->k_row_bytes * out->slots;
  out->v_head_stride_bytes = out->v_row_bytes * out->slots;
  out->k_seq_stride_bytes = out->k_head_stride_bytes * cfg->n_kv_heads;
  out->v_seq_stride_bytes = out->v_head_stride_bytes * cfg->n_kv_heads;
  out->k_cache_bytes = out->k_seq_stride_bytes * cfg->max_seqs;
  out->v_cache_bytes = cfg->v_aliases_k ? 0 : out->v_seq_stride_bytes * cfg->max_seqs;
  return SNAP_OK;
}

int64_t snap_compress_workspace_bytes(const snap_config_t* cfg, const int32_t* cu_seqlens_host,
                                      int32_t n_seq) {
  int rc = validate(cfg);
  if (rc != SNAP_OK) return rc;
  rc = check_cu(cu_seqlens_host, n_seq);
  if (rc != SNAP_OK) return rc;
  const Shape s = make_shape(cfg);
  size_t worst = 0;
  for (int first = 0; first < n_seq; first += kMaxBatchSeqs) {
    const int n = n_seq - first < kMaxBatchSeqs ? n_seq - first : kMaxBatchSeqs;
    const ChunkPlan p = plan_chunk(cfg->dtype, s, cu_seqlens_host, first, n);
    worst = p.bytes > worst ? p.bytes : worst;
  }
  return (int64_t)(idx_bytes(s, n_seq) + worst + 256);
}

int64_t snap_decode_workspace_bytes(const snap_config_t* cfg, int32_t n_active) {
  const int rc = validate(cfg);
  if (rc != SNAP_OK) return rc;
  if (n_active < 0) return SNAP_ERR_INVALID_ARG;
  const Shape s = make_shape(cfg);
  const DecodePlan p = plan_decode(cfg->dtype, s, n_active);
  return (int64_t)(p.floats * sizeof(float) + 256);
}

int snap_compress(const snap_config_t* cfg, const snap_layout_t* layout, const void* q_obs_dev,
                  const void* k_dev, int64_t k_token_stride, int64_t k_head_stride,
                  const void* v_dev, int64_t v_token_stride, int64_t v_head_stride,
                  const int32_t* cu_seqlens_host, const int32_t* slot_ids_host, int32_t n_seq,
                  void* k_cache_dev, void* v_cache_dev, int32_t* seq_len_dev,
                  int32_t* valid_topk_dev, int32_t* topk_idx_dev, void* workspace_dev,
                  size_t workspace_bytes, uint32_t* status_dev, void* cuda_stream) {
  return snap_compress_with_row_stats(cfg, layout, q_obs_dev, nullptr, k_dev, k_token_stride, k_head_stride, v_dev,
                                      v_token_stride, v_head_stride, cu_seqlens_host, slot_ids_host, n_seq, k_cache_dev,
                                      v_cache_dev, seq_len_dev, valid_topk_dev, topk_idx_dev, workspace_dev,
                                      workspace_bytes, status_dev, cuda_stream);
}

int snap_prefill_attn(const snap_config_t* cfg, const void* q_dev,
                      const void* k_dev, int64_t k_token_stride, int64_t k_head_stride,
                      const void* v_dev, int64_t v_token_stride, int64_t v_head_stride,
                      const int32_t* cu_seqlens_host, int32_t n_seq, void* out_dev, float* row_mu_dev,
                      uint32_t* status_dev, void* cuda_stream) {
  int rc = validate(cfg);
  if (rc != SNAP_OK) return rc;
  rc = check_cu(cu_seqlens_host, n_seq);
  if (rc != SNAP_OK) return rc;
  const Shape s = make_shape(cfg);
  if (n_seq == 0 || cu_seqlens_host[n_seq] == cu_seqlens_host[0]) return SNAP_OK;
  if (!q_dev || !k_dev || !out_dev || (!cfg->v_aliases_k && !v_dev)) return SNAP_ERR_NULL_POINTER;
  if (misaligned(q_dev, k_dev, v_dev, out_dev)) return SNAP_ERR_INVALID_ARG;
  const int eb = elt_bytes(cfg->dtype);
  if ((k_token_stride * eb) % 16 || (k_head_stride * eb) % 16 || k_token_stride < s.d_qk) return SNAP_ERR_INVALID_ARG;
  if (!cfg->v_aliases_k && ((v_token_stride * eb) % 16 || (v_head_stride * eb) % 16 || v_token_stride < s.d_v))
    return SNAP_ERR_INVALID_ARG;
  // option SNAP_OPT_PREFILL_KERNEL = 1 forces the portable kernel (testing aid)
  const bool tensor_path = prefill_attn_supported(cfg->dtype, s) && option(SNAP_OPT_PREFILL_KERNEL) != 1;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  KVSource src;
  src.k = k_dev; src.v = v_dev;
  src.k_tok_stride = k_token_stride; src.k_head_stride = k_head_stride;
  src.v_tok_stride = v_token_stride; src.v_head_stride = v_head_stride;
  for (int first = 0; first < n_seq; first += kMaxBatchSeqs) {
    const int n = n_seq - first < kMaxBatchSeqs ? n_seq - first : kMaxBatchSeqs;
    SeqBatch b;
    std::memset(&b, 0, sizeof(b));
    b.n = n; b.first_seq = first;
    for (int i = 0; i < n; ++i) {
      b.tok_off[i] = cu_seqlens_host[first + i];
      b.len[i] = cu_seqlens_host[first + i + 1] - cu_seqlens_host[first + i];
    }
    const cudaError_t e = tensor_path ? launch_prefill_attn(s, b, q_dev, src, out_dev, row_mu_dev, status_dev, st)
                                      : launch_prefill_generic(cfg->dtype, s, b, q_dev, src, out_dev, row_mu_dev, st);
    if (e != cudaSuccess) return SNAP_ERR_CUDA;
  }
  return SNAP_OK;
}

int snap_compress_with_row_stats(const snap_config_t* cfg, const snap_layout_t* layout, const void* q_obs_dev,
                                 const float* row_mu_dev,
                                 const void* k_dev, int64_t k_token_stride, int64_t k_head_stride,
                                 const void* v_dev, int64_t v_token_stride, int64_t v_head_stride,
                                 const int32_t* cu_seqlens_host, const int32_t* slot_ids_host, int32_t n_seq,
                                 void* k_cache_dev, void* v_cache_dev, int32_t* seq_len_dev,
                                 int32_t* valid_topk_dev, int32_t* topk_idx_dev, void* workspace_dev,
                                 size_t workspace_bytes, uint32_t* status_dev, void* cuda_stream) {
  int rc = validate(cfg);
  if (rc != SNAP_OK) return rc;
  if (!layout || !slot_ids_host) return SNAP_ERR_NULL_POINTER;
  rc = check_cu(cu_seqlens_host, n_seq);
  if (rc != SNAP_OK) return rc;
  if (n_seq == 0) return SNAP_OK;
  if (!k_dev || !k_cache_dev || !seq_len_dev || !valid_topk_dev) return SNAP_ERR_NULL_POINTER;
  if (!cfg->v_aliases_k && (!v_dev || !v_cache_dev)) return SNAP_ERR_NULL_POINTER;
  if (misaligned(q_obs_dev, k_dev, v_dev, k_cache_dev, v_cache_dev, workspace_dev)) return SNAP_ERR_INVALID_ARG;
  const Shape s = make_shape(cfg);
  if (layout->slots != s.Sc) return SNAP_ERR_INVALID_ARG;
  const int eb = elt_bytes(cfg->dtype);
  if ((k_token_stride * eb) % 16 || (k_head_stride * eb) % 16 || k_token_stride < s.d_qk)
    return SNAP_ERR_INVALID_ARG;
  if (!cfg->v_aliases_k && ((v_token_stride * eb) % 16 || (v_head_stride * eb) % 16 || v_token_stride < s.d_v))
    return SNAP_ERR_INVALID_ARG;
  {
    std::vector<char> seen((size_t)cfg->max_seqs, 0);
    for (int i = 0; i < n_seq; ++i) {
      const int sl = slot_ids_host[i];
      if (sl < 0 || sl >= cfg->max_seqs || seen[sl]) return SNAP_ERR_INVALID_ARG;
      seen[sl] = 1;
    }
  }
  const int64_t need = snap_compress_workspace_bytes(cfg, cu_seqlens_host, n_seq);
  if (need < 0) return (int)need;
  bool any_scored = false;
  for (int i = 0; i < n_seq; ++i) {
    const int L = cu_seqlens_host[i + 1] - cu_seqlens_host[i];
    if (s.K > 0 && L - s.Ls - s.Lr > s.K) any_scored = true;
  }
  if (any_scored && !q_obs_dev) return SNAP_ERR_NULL_POINTER;
  if ((any_scored || !topk_idx_dev) && s.K > 0) {
    if (!workspace_dev) return SNAP_ERR_NULL_POINTER;
    if (workspace_bytes < (size_t)need) return SNAP_ERR_WORKSPACE_TOO_SMALL;
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace_dev);
  int* idx = topk_idx_dev ? topk_idx_dev : reinterpret_cast<int*>(ws);
  char* chunk_ws = ws ? ws + idx_bytes(s, n_seq) : nullptr;

  KVSource src;
  src.k = k_dev; src.v = cfg->v_aliases_k ? nullptr : v_dev;
  src.k_tok_stride = k_token_stride; src.k_head_stride = k_head_stride;
  src.v_tok_stride = v_token_stride; src.v_head_stride = v_head_stride;

  for (int first = 0; first < n_seq; first += kMaxBatchSeqs) {
    const int n = n_seq - first < kMaxBatchSeqs ? n_seq - first : kMaxBatchSeqs;
    const ChunkPlan p = plan_chunk(cfg->dtype, s, cu_seqlens_host, first, n);
    SeqBatch b;
    std::memset(&b, 0, sizeof(b));
    b.n = n; b.first_seq = first;
    for (int i = 0; i < n; ++i) {
      b.tok_off[i] = cu_seqlens_host[first + i];
      b.len[i] = cu_seqlens_host[first + i + 1] - cu_seqlens_host[first + i];
      b.slot[i] = slot_ids_host[first + i];
      b.score_idx[i] = -1;
      if (s.K > 0 && b.len[i] - s.Ls - s.Lr > s.K) {
        b.score_idx[i] = b.n_scored;
        b.seq_of_score[b.n_scored++] = i;
      }
    }
    ScoreBuffers buf;
    std::memset(&buf, 0, sizeof(buf));
    if (p.n_scored > 0) {
      buf.part_stats = reinterpret_cast<float2*>(chunk_ws + p.part_off);
      buf.stats = reinterpret_cast<float2*>(chunk_ws + p.stats_off);
      buf.C = reinterpret_cast<float*>(chunk_ws + p.c_off);
      buf.P = reinterpret_cast<float*>(chunk_ws + p.p_off);
      buf.c_stride = p.c_stride; buf.nsplit = p.nsplit; buf.chunk_tiles = p.chunk_tiles;
      buf.ext_mu = row_mu_dev;
      if (p.ref_cap > 0) {
        buf.ref.head = reinterpret_cast<RefineHead*>(chunk_ws + p.ref_head_off);
        buf.ref.band = reinterpret_cast<BandEntry*>(chunk_ws + p.ref_band_off);
        buf.ref.part = reinterpret_cast<double*>(chunk_ws + p.ref_part_off);
        buf.ref.mu64 = row_mu_dev ? nullptr : reinterpret_cast<double*>(chunk_ws + p.ref_mu_off);
        buf.ref.lists = reinterpret_cast<int*>(chunk_ws + p.ref_lists_off);
        buf.ref.cap = p.ref_cap; buf.ref.chunks = p.ref_chunks; buf.ref.rel = p.ref_rel;
        buf.ref.stats_natural = !use_umma(cfg->dtype, s) && !use_umma_wide(cfg->dtype, s) && !use_mma(cfg->dtype, s);
      }
      const cudaError_t e = use_umma(cfg->dtype, s)  ? launch_score_umma(s, b, q_obs_dev, src, buf, status_dev, st)
                            : use_umma_wide(cfg->dtype, s)
                                ? launch_score_umma_wide(s, b, q_obs_dev, src, buf,
                                                         reinterpret_cast<float*>(chunk_ws + p.cpart_off), status_dev, st)
                            : use_mma(cfg->dtype, s) ? launch_score_mma(s, b, q_obs_dev, src, buf, st)
                                                     : launch_score_simt(cfg->dtype, s, b, q_obs_dev, src, buf, st);
      if (e != cudaSuccess) return SNAP_ERR_CUDA;
    }
    if (launch_pool_topk(s, b, buf, idx, status_dev, st) != cudaSuccess) return SNAP_ERR_CUDA;
    if (launch_topk_refine(cfg->dtype, s, b, q_obs_dev, src, buf, status_dev, sm_count(), st) != cudaSuccess)
      return SNAP_ERR_CUDA;
    if (launch_gather(cfg->dtype, s, b, src, idx, k_cache_dev, v_cache_dev, seq_len_dev,
                      valid_topk_dev, status_dev, st, &buf) != cudaSuccess)
      return SNAP_ERR_CUDA;
  }
  return SNAP_OK;
}

int snap_append_kv(const snap_config_t* cfg, const snap_layout_t* layout, const void* k_new_dev,
                   const void* v_new_dev, const int32_t* slot_ids_dev, int32_t n_active,
                   void* k_cache_dev, void* v_cache_dev, int32_t* seq_len_dev,
                   uint32_t* status_dev, void* cuda_stream) {
  const int rc = validate(cfg);
  if (rc != SNAP_OK) return rc;
  if (!layout) return SNAP_ERR_NULL_POINTER;
  if (n_active < 0) return SNAP_ERR_INVALID_ARG;
  if (n_active == 0) return SNAP_OK;
  if (!k_new_dev || !slot_ids_dev || !k_cache_dev || !seq_len_dev) return SNAP_ERR_NULL_POINTER;
  if (!cfg->v_aliases_k && (!v_new_dev || !v_cache_dev)) return SNAP_ERR_NULL_POINTER;
  if (misaligned(k_new_dev, v_new_dev, k_cache_dev, v_cache_dev)) return SNAP_ERR_INVALID_ARG;
  const Shape s = make_shape(cfg);
  if (layout->slots != s.Sc) return SNAP_ERR_INVALID_ARG;
  if (launch_append(cfg->dtype, s, k_new_dev, v_new_dev, slot_ids_dev, n_active, k_cache_dev,
                    v_cache_dev, seq_len_dev, status_dev,
                    static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
    return SNAP_ERR_CUDA;
  return SNAP_OK;
}

int snap_decode_attn(const snap_config_t* cfg, const snap_layout_t* layout, const void* q_dev,
                     const void* k_new_dev, const void* v_new_dev, const int32_t* slot_ids_dev,
                     int32_t n_active, void* k_cache_dev, void* v_cache_dev, int32_t* seq_len_dev,
                     const int32_t* valid_topk_dev, void* out_dev, void* workspace_dev,
                     size_t workspace_bytes, uint32_t* status_dev, void* cuda_stream) {
  return decode_step_with_scratch(cfg, layout, q_dev, k_new_dev, v_new_dev, slot_ids_dev, n_active, k_cache_dev,
                                  v_cache_dev, seq_len_dev, valid_topk_dev, out_dev, static_cast<float*>(workspace_dev),
                                  workspace_bytes, 256, SNAP_ERR_WORKSPACE_TOO_SMALL, status_dev, cuda_stream);
}

// Several query tokens per sequence in one step.  The tensor-core kernel for bf16 heads serves
// them in one pass over the cache (the tokens' heads share the N side of its MMAs, so
// q_len * group <= 8); every other shape is served as the definition reads: q_len single steps,
// each token's rows staged densely in the workspace by strided device-to-device copies.
static int multi_check(const Shape& s, int q_len) {
  return q_len < 1 || q_len > s.Lr ? SNAP_ERR_INVALID_ARG : SNAP_OK;
}
// Tokens per launch of the tensor-core grouped-query kernel: its MMA columns hold (token, head)
// pairs, eight or sixteen of them, so 16 / g tokens go in one pass and a longer step takes several
// passes, each reading its tokens' rows in place.  0: the layout is served by other kernels.
static int multi_tokens_per_pass(const snap_config_t* cfg, const Shape& s, int q_len) {
  if (!decode_use_gqa_mma(cfg->dtype, s) || s.g > 16) return 0;
  const int t = 16 / s.g;
  return t < q_len ? t : q_len;
}

// Dense staging of one token's rows for the step-wise path: q, k_new, v_new, out.
struct StepStage { size_t q_row, k_row, v_row, o_row, q_off, k_off, v_off, o_off, bytes; };
static StepStage step_stage(const snap_config_t* cfg, const Shape& s, int n_active) {
  StepStage t;
  const size_t eb = (size_t)elt_bytes(cfg->dtype), n = (size_t)(n_active > 0 ? n_active : 0);
  t.q_row = (size_t)s.Hq * s.d_qk * eb;
  t.k_row = (size_t)s.Hkv * s.d_qk * eb;
  t.v_row = s.v_aliases_k ? 0 : (size_t)s.Hkv * s.d_v * eb;
  t.o_row = (size_t)s.Hq * s.d_v * eb;
  size_t off = 0;
  t.q_off = off; off += align_up(n * t.q_row);
  t.k_off = off; off += align_up(n * t.k_row);
  t.v_off = off; off += align_up(n * t.v_row);
  t.o_off = off; off += align_up(n * t.o_row);
  t.bytes = off;
  return t;
}

int64_t snap_decode_multi_workspace_bytes(const snap_config_t* cfg, int32_t n_active, int32_t q_len) {
  const int rc = validate(cfg);
  if (rc != SNAP_OK) return rc;
  if (n_active < 0) return SNAP_ERR_INVALID_ARG;
  const Shape s = make_shape(cfg);
  const int mc = multi_check(s, q_len);
  if (mc != SNAP_OK) return mc;
  if (const int tpp = multi_tokens_per_pass(cfg, s, q_len)) {
    const int nsplit = decode_gqa_mma_nsplit(s, n_active > 0 ? n_active : 1, sm_count());
    return (int64_t)(decode_gqa_mma_partial_floats(s, n_active * tpp, nsplit) * sizeof(float) + 256);
  }
  const int64_t single = snap_decode_workspace_bytes(cfg, n_active);
  if (single < 0) return single;
  return (int64_t)step_stage(cfg, s, n_active).bytes + single;
}

// ---- per-step block top-K over the third section (block_topk.cu) ----

static int blocks_check(const snap_config_t* cfg, const Shape& s, int block_tokens) {
  if (block_tokens < 1) return SNAP_ERR_INVALID_ARG;
  if (!block_topk_supported(cfg->dtype, s, block_tokens) || !decode_use_gqa_mma(cfg->dtype, s)) return SNAP_ERR_UNSUPPORTED;
  return SNAP_OK;
}
// the cache the decode kernel's split rule should assume: the low section plus the visited blocks
static Shape blocks_shape(Shape s, int block_tokens, int n_blocks) {
  const long long rows = (long long)n_blocks * block_tokens;
  s.K = rows < s.K ? (int)rows : s.K;
  s.Sc = s.Ls + s.Lr + s.K;
  return s;
}

int64_t snap_block_stats_bytes(const snap_config_t* cfg, int32_t block_tokens) {
  const int rc = validate(cfg);
  if (rc != SNAP_OK) return rc;
  const Shape s = make_shape(cfg);
  const int bc = blocks_check(cfg, s, block_tokens);
  if (bc != SNAP_OK) return bc;
  return (int64_t)s.max_seqs * s.Hkv * block_count_max(s, block_tokens) * 2 * s.d_qk * elt_bytes(cfg->dtype);
}

int snap_block_stats(const snap_config_t* cfg, const snap_layout_t* layout, const int32_t* slot_ids_dev, int32_t n_seqs,
                     const void* k_cache_dev, const int32_t* valid_topk_dev, int32_t block_tokens, void* stats_dev,
                     uint32_t* status_dev, void* cuda_stream) {
  const int rc = validate(cfg);
  if (rc != SNAP_OK) return rc;
  if (!layout) return SNAP_ERR_NULL_POINTER;
  if (n_seqs < 0) return SNAP_ERR_INVALID_ARG;
  const Shape s = make_shape(cfg);
  const int bc = blocks_check(cfg, s, block_tokens);
  if (bc != SNAP_OK) return bc;
  if (layout->slots != s.Sc) return SNAP_ERR_INVALID_ARG;
  if (n_seqs == 0) return SNAP_OK;
  if (!slot_ids_dev || !k_cache_dev || !valid_topk_dev || !stats_dev) return SNAP_ERR_NULL_POINTER;
  if (misaligned(k_cache_dev, stats_dev)) return SNAP_ERR_INVALID_ARG;
  const cudaError_t e = launch_block_stats(s, block_tokens, slot_ids_dev, n_seqs, k_cache_dev, valid_topk_dev, stats_dev,
                                           status_dev, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? SNAP_OK : SNAP_ERR_CUDA;
}

int snap_block_select(const snap_config_t* cfg, const snap_layout_t* layout, const void* q_dev, const int32_t* slot_ids_dev,
                      int32_t n_active, const void* stats_dev, const int32_t* valid_topk_dev, int32_t block_tokens,
                      int32_t n_blocks, int32_t* block_idx_dev, int32_t* n_selected_dev, void* workspace_dev,
                      size_t workspace_bytes, uint32_t* status_dev, void* cuda_stream) {
  const int rc = validate(cfg);
  if (rc != SNAP_OK) return rc;
  if (!layout) return SNAP_ERR_NULL_POINTER;
  if (n_active < 0 || n_blocks < 1) return SNAP_ERR_INVALID_ARG;
  const Shape s = make_shape(cfg);
  const int bc = blocks_check(cfg, s, block_tokens);
  if (bc != SNAP_OK) return bc;
  if (layout->slots != s.Sc) return SNAP_ERR_INVALID_ARG;
  if (n_active == 0) return SNAP_OK;
  if (!q_dev || !slot_ids_dev || !stats_dev || !valid_topk_dev || !block_idx_dev || !n_selected_dev || !workspace_dev)
    return SNAP_ERR_NULL_POINTER;
  if (misaligned(q_dev, stats_dev, workspace_dev)) return SNAP_ERR_INVALID_ARG;
  if (workspace_bytes < block_select_scratch_bytes(s, block_tokens, n_active)) return SNAP_ERR_WORKSPACE_TOO_SMALL;
  const cudaError_t e = launch_block_select(s, block_tokens, n_blocks, q_dev, slot_ids_dev, n_active, stats_dev, valid_topk_dev,
                                            block_idx_dev, n_selected_dev, workspace_dev, status_dev,
                                            static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? SNAP_OK : SNAP_ERR_CUDA;
}

int64_t snap_block_select_workspace_bytes(const snap_config_t* cfg, int32_t n_active, int32_t block_tokens) {
  const int rc = validate(cfg);
  if (rc != SNAP_OK) return rc;
  if (n_active < 0) return SNAP_ERR_INVALID_ARG;
  const Shape s = make_shape(cfg);
  const int bc = blocks_check(cfg, s, block_tokens);
  if (bc != SNAP_OK) return bc;
  return (int64_t)block_select_scratch_bytes(s, block_tokens, n_active);
}

int64_t snap_decode_blocks_workspace_bytes(const snap_config_t* cfg, int32_t n_active, int32_t block_tokens, int32_t n_blocks) {
  const int rc = validate(cfg);
  if (rc != SNAP_OK) return rc;
  if (n_active < 0 || n_blocks < 1) return SNAP_ERR_INVALID_ARG;
  const Shape s = make_shape(cfg);
  const int bc = blocks_check(cfg, s, block_tokens);
  if (bc != SNAP_OK) return bc;
  const int nsplit = decode_gqa_mma_nsplit(blocks_shape(s, block_tokens, n_blocks), n_active > 0 ? n_active : 1, sm_count());
  return (int64_t)(decode_gqa_mma_partial_floats(s, n_active, nsplit) * sizeof(float) + 256);
}

int snap_decode_attn_blocks(const snap_config_t* cfg, const snap_layout_t* layout, const void* q_dev, const void* k_new_dev,
                            const void* v_new_dev, const int32_t* slot_ids_dev, int32_t n_active, void* k_cache_dev,
                            void* v_cache_dev, int32_t* seq_len_dev, const int32_t* valid_topk_dev, int32_t block_tokens,
                            int32_t n_blocks, const int32_t* block_idx_dev, const int32_t* n_selected_dev, void* out_dev,
                            void* workspace_dev, size_t workspace_bytes, uint32_t* status_dev, void* cuda_stream) {
  const int rc = validate(cfg);
  if (rc != SNAP_OK) return rc;
  if (!layout) return SNAP_ERR_NULL_POINTER;
  if (n_active < 0 || n_blocks < 1) return SNAP_ERR_INVALID_ARG;
  const Shape s = make_shape(cfg);
  const int bc = blocks_check(cfg, s, block_tokens);
  if (bc != SNAP_OK) return bc;
  if (layout->slots != s.Sc) return SNAP_ERR_INVALID_ARG;
  if (n_active == 0) return SNAP_OK;
  if (!q_dev || !slot_ids_dev || !k_cache_dev || !v_cache_dev || !seq_len_dev || !valid_topk_dev || !block_idx_dev ||
      !n_selected_dev || !out_dev || !workspace_dev)
    return SNAP_ERR_NULL_POINTER;
  if (k_new_dev && !v_new_dev) return SNAP_ERR_NULL_POINTER;
  if (misaligned(q_dev, k_new_dev, v_new_dev, k_cache_dev, v_cache_dev, out_dev, workspace_dev)) return SNAP_ERR_INVALID_ARG;
  const int64_t need = snap_decode_blocks_workspace_bytes(cfg, n_active, block_tokens, n_blocks);
  if (need < 0) return (int)need;
  if (workspace_bytes < (size_t)need) return SNAP_ERR_WORKSPACE_TOO_SMALL;
  const int nsplit = decode_gqa_mma_nsplit(blocks_shape(s, block_tokens, n_blocks), n_active, sm_count());
  const cudaError_t e = launch_decode_gqa_mma(s, q_dev, k_new_dev, v_new_dev, slot_ids_dev, n_active, k_cache_dev, v_cache_dev,
                                              seq_len_dev, valid_topk_dev, out_dev, static_cast<float*>(workspace_dev), nsplit,
                                              status_dev, static_cast<cudaStream_t>(cuda_stream), 1, 0, 0, block_idx_dev,
                                              n_selected_dev, n_blocks, block_tokens);
  return e == cudaSuccess ? SNAP_OK : SNAP_ERR_CUDA;
}

int snap_decode_attn_multi(const snap_config_t* cfg, const snap_layout_t* layout, const void* q_dev,
                           const void* k_new_dev, const void* v_new_dev, const int32_t* slot_ids_dev,
                           int32_t n_active, int32_t q_len, void* k_cache_dev, void* v_cache_dev,
                           int32_t* seq_len_dev, const int32_t* valid_topk_dev, void* out_dev,
                           void* workspace_dev, size_t workspace_bytes, uint32_t* status_dev, void* cuda_stream) {
  const int rc = validate(cfg);
  if (rc != SNAP_OK) return rc;
  if (!layout) return SNAP_ERR_NULL_POINTER;
  if (n_active < 0) return SNAP_ERR_INVALID_ARG;
  const Shape s = make_shape(cfg);
  const int mc = multi_check(s, q_len);
  if (mc != SNAP_OK) return mc;
  if (n_active == 0) return SNAP_OK;
  if (!q_dev || !k_new_dev || !slot_ids_dev || !k_cache_dev || !seq_len_dev || !valid_topk_dev || !out_dev ||
      !workspace_dev)
    return SNAP_ERR_NULL_POINTER;
  if (!s.v_aliases_k && (!v_new_dev || !v_cache_dev)) return SNAP_ERR_NULL_POINTER;
  if (misaligned(q_dev, k_new_dev, v_new_dev, k_cache_dev, v_cache_dev, out_dev, workspace_dev)) return SNAP_ERR_INVALID_ARG;
  if (layout->slots != s.Sc) return SNAP_ERR_INVALID_ARG;
  const int64_t need = snap_decode_multi_workspace_bytes(cfg, n_active, q_len);
  if (need < 0) return (int)need;
  if (workspace_bytes < (size_t)need) return SNAP_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (const int tpp = multi_tokens_per_pass(cfg, s, q_len)) {
    const int nsplit = decode_gqa_mma_nsplit(s, n_active, sm_count());
    for (int u0 = 0; u0 < q_len; u0 += tpp) {
      const int t = q_len - u0 < tpp ? q_len - u0 : tpp;
      if (launch_decode_gqa_mma(s, q_dev, k_new_dev, v_new_dev, slot_ids_dev, n_active, k_cache_dev, v_cache_dev, seq_len_dev,
                                valid_topk_dev, out_dev, static_cast<float*>(workspace_dev), nsplit, status_dev, st, t, q_len,
                                u0) != cudaSuccess)
        return SNAP_ERR_CUDA;
    }
    return SNAP_OK;
  }
  // the streamed latent kernel reads token u of every sequence in place (strided tensor map, strided rows):
  // q_len single steps with no staging copies.  (One launch over (sequence, token) was tried: with the 8 sequences
  // of the latent benchmark shape the grid needs two waves and two tokens took 140 us against 2 x 54.)
  {
    const DecodePlan p = plan_decode(cfg->dtype, s, n_active);
    if (p.mla_stream) {
      for (int u = 0; u < q_len; ++u)
        if (launch_decode_mla_stream(s, q_dev, k_new_dev, slot_ids_dev, n_active, k_cache_dev, seq_len_dev, valid_topk_dev,
                                     out_dev, static_cast<float*>(workspace_dev), p.nsplit, status_dev, st, q_len, u) != cudaSuccess)
          return SNAP_ERR_CUDA;
      return SNAP_OK;
    }
  }
  // q_len single steps: token u of every sequence is gathered into dense rows, attended, and its
  // output scattered back
  const StepStage t = step_stage(cfg, s, n_active);
  char* ws = static_cast<char*>(workspace_dev);
  char* single_ws = ws + t.bytes;
  const size_t single_bytes = workspace_bytes - t.bytes;
  auto gather = [&](char* dst, const void* src, size_t row, int u) {
    return row == 0 ? cudaSuccess
                    : cudaMemcpy2DAsync(dst, row, static_cast<const char*>(src) + (size_t)u * row, (size_t)q_len * row, row,
                                        (size_t)n_active, cudaMemcpyDeviceToDevice, st);
  };
  for (int u = 0; u < q_len; ++u) {
    if (gather(ws + t.q_off, q_dev, t.q_row, u) != cudaSuccess || gather(ws + t.k_off, k_new_dev, t.k_row, u) != cudaSuccess ||
        gather(ws + t.v_off, v_new_dev, t.v_row, u) != cudaSuccess)
      return SNAP_ERR_CUDA;
    const int r = snap_decode_attn(cfg, layout, ws + t.q_off, ws + t.k_off, s.v_aliases_k ? nullptr : ws + t.v_off,
                                   slot_ids_dev, n_active, k_cache_dev, v_cache_dev, seq_len_dev, valid_topk_dev,
                                   ws + t.o_off, single_ws, single_bytes, status_dev, cuda_stream);
    if (r != SNAP_OK) return r;
    if (cudaMemcpy2DAsync(static_cast<char*>(out_dev) + (size_t)u * t.o_row, (size_t)q_len * t.o_row, ws + t.o_off, t.o_row,
                          t.o_row, (size_t)n_active, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
      return SNAP_ERR_CUDA;
  }
  return SNAP_OK;
}

}  // extern "C"
