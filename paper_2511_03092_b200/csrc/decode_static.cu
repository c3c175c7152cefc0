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

// Per-device set-up on first use, with that device current: resolve the array's device address.
int static_scratch(float** ptr) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SNAP_ERR_CUDA;
  if (!g_scratch_ptr[dev]) {
    float* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_partials) != cudaSuccess || !p)
      return SNAP_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  *ptr = g_scratch_ptr[dev];
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
  float* scratch = nullptr;
  const int src = static_scratch(&scratch);
  if (src != SNAP_OK) return src;
  // Everything else -- validation, the choice of kernel and split count, the launches -- is the
  // body of snap_decode_attn, so the two entry points cannot drift apart: the latent layout runs
  // its own kernels here too.
  return decode_step_with_scratch(cfg, layout, q_dev, k_new_dev, v_new_dev, slot_ids_dev, n_active, k_cache_dev,
                                  v_cache_dev, seq_len_dev, valid_topk_dev, out_dev, scratch,
                                  SNAP_STATIC_SCRATCH_BYTES, 0, SNAP_ERR_STATIC_SCRATCH_EXCEEDED, status_dev,
                                  cuda_stream);
}
