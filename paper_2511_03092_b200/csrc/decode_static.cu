// snap_decode_attn_static: the decode step for callers that cannot provide scratch memory.
//
// Some hosts of this library never get to call cudaMalloc at the point where a decode step is
// issued: a serving loop whose memory pool was carved up and frozen at start-up, a plugin that
// runs inside another framework's stream callback or graph-building phase, code running under
// a strict out-of-memory policy where any late allocation is a failure.  snap_decode_attn
// needs a scratch buffer for the per-split partial results, and those callers have nowhere to
// take it from.  This variant keeps that scratch in a fixed array inside the library instead.
//
// Consequences, all documented in snapstream.h as well:
//   * the array is SNAP_STATIC_SCRATCH_BYTES large and every GPU that loads the library holds
//     it until the process exits;
//   * a problem whose partial results do not fit is refused (SNAP_ERR_STATIC_SCRATCH_EXCEEDED),
//     nothing is launched;
//   * all calls share the one array, so two calls that may overlap on the GPU (different
//     streams, no dependency) race with each other -- serialise them;
//   * the array keeps whatever the previous call left; the split kernel overwrites every
//     partial that the merge kernel later reads, so nothing needs clearing between calls;
//   * the device address of the array is looked up on the first call on each device (one
//     cudaGetSymbolAddress, no allocation).  Make that first call outside any stream capture.
#include "snap_internal.cuh"

namespace snap {
namespace {

constexpr size_t kStaticFloats = SNAP_STATIC_SCRATCH_BYTES / sizeof(float);

// The scratch itself.  In host code this name is only a handle for the runtime, not an address
// the GPU can use; the usable address comes from cudaGetSymbolAddress below.
static __device__ __align__(256) float g_static_partials[kStaticFloats];

float* g_scratch_ptr[kMaxDevices] = {};
int g_sm_count[kMaxDevices] = {};

// Per-device set-up on first use, with that device current: resolve the array's device address.
int static_scratch(float** ptr, int* sms) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SNAP_ERR_CUDA;
  if (!g_scratch_ptr[dev]) {
    float* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_partials) != cudaSuccess || !p)
      return SNAP_ERR_CUDA;
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1)
      return SNAP_ERR_CUDA;
    g_sm_count[dev] = n;
    g_scratch_ptr[dev] = p;
  }
  *ptr = g_scratch_ptr[dev];
  *sms = g_sm_count[dev];
  return SNAP_OK;
}

}  // namespace
}  // namespace snap

using namespace snap;

extern "C" int snap_decode_attn_static(const snap_config_t* cfg, const snap_layout_t* layout,
                                       const void* q_dev, const void* k_new_dev, const void* v_new_dev,
                                       const int32_t* slot_ids_dev, int32_t n_active,
                                       void* k_cache_dev, void* v_cache_dev, int32_t* seq_len_dev,
                                       const int32_t* valid_topk_dev, void* out_dev,
                                       uint32_t* status_dev, void* cuda_stream) {
  // Validation of the configuration is shared with the other entry points through the layout
  // routine (pure host arithmetic, allocates nothing).
  snap_layout_t lay;
  const int rc = snap_cache_layout(cfg, &lay);
  if (rc != SNAP_OK) return rc;
  if (!layout) return SNAP_ERR_NULL_POINTER;
  if (n_active < 0 || layout->slots != lay.slots) return SNAP_ERR_INVALID_ARG;
  if (n_active == 0) return SNAP_OK;
  if (!q_dev || !slot_ids_dev || !k_cache_dev || !seq_len_dev || !valid_topk_dev || !out_dev)
    return SNAP_ERR_NULL_POINTER;
  if (!cfg->v_aliases_k && !v_cache_dev) return SNAP_ERR_NULL_POINTER;
  if (k_new_dev && !cfg->v_aliases_k && !v_new_dev) return SNAP_ERR_NULL_POINTER;

  Shape s;
  s.Hq = cfg->n_q_heads; s.Hkv = cfg->n_kv_heads; s.g = s.Hq / s.Hkv; s.d_qk = cfg->d_qk; s.d_v = cfg->d_v;
  s.Ls = cfg->l_sink; s.Lr = cfg->l_recent; s.K = cfg->topk; s.Lo = cfg->l_obs; s.w = cfg->pool_kernel;
  s.pool_mode = cfg->pool_mode; s.v_aliases_k = cfg->v_aliases_k; s.Sc = lay.slots;
  s.max_seqs = cfg->max_seqs; s.scale = cfg->softmax_scale;

  float* scratch = nullptr;
  int sms = 0;
  const int src = static_scratch(&scratch, &sms);
  if (src != SNAP_OK) return src;

  const bool gqa_mma = decode_use_gqa_mma(cfg->dtype, s);
  const bool gqa = gqa_mma || decode_gqa_supported(cfg->dtype, s);
  const int nsplit = gqa_mma ? decode_gqa_mma_nsplit(s, n_active, sms)
                     : gqa   ? decode_gqa_nsplit(s, n_active, sms)
                             : decode_generic_nsplit(s, n_active, sms);
  const size_t need = gqa_mma ? decode_gqa_mma_partial_floats(s, n_active, nsplit)
                      : gqa   ? decode_gqa_partial_floats(s, n_active, nsplit)
                              : decode_partial_floats(s, n_active, nsplit);
  if (need > kStaticFloats) return SNAP_ERR_STATIC_SCRATCH_EXCEEDED;

  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e;
  if (gqa_mma)
    e = launch_decode_gqa_mma(s, q_dev, k_new_dev, v_new_dev, slot_ids_dev, n_active, k_cache_dev,
                              v_cache_dev, seq_len_dev, valid_topk_dev, out_dev, scratch, nsplit,
                              status_dev, st);
  else if (gqa)
    e = launch_decode_gqa(s, q_dev, k_new_dev, v_new_dev, slot_ids_dev, n_active, k_cache_dev,
                          v_cache_dev, seq_len_dev, valid_topk_dev, out_dev, scratch, nsplit,
                          status_dev, st);
  else
    e = launch_decode_generic(cfg->dtype, s, q_dev, k_new_dev, v_new_dev, slot_ids_dev, n_active,
                              k_cache_dev, v_cache_dev, seq_len_dev, valid_topk_dev, out_dev,
                              scratch, nsplit, status_dev, st);
  return e == cudaSuccess ? SNAP_OK : SNAP_ERR_CUDA;
}
