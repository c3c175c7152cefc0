// snap_append_kv_concat: the slice-and-concatenate cache update that Section 3.2.1 argues
// against, kept as a measured baseline for the ring buffer of Eq. 3.
//
// The recent window is held in position order.  Once it is full, a new token drops the oldest
// window row, moves every other window row down by one and goes last; because a concatenation
// produces a new tensor, the whole cache [sink | window | top-K] is rewritten into a second
// buffer each step.  On a GPU this parallelises without trouble -- one thread per 16 bytes of
// the output -- so what it costs is traffic: the cache is read once and written once per
// decoded token, where the ring buffer writes one row.
#include "snap_internal.cuh"

namespace snap {
namespace {

constexpr int NT = 256, ROWS = 16;

struct ConcatArgs {
  const char* k_new; const char* v_new;
  const char* kin; const char* vin;
  char* kout; char* vout;
  long long k_seq_b, k_head_b, v_seq_b, v_head_b;
  int k_row_b, v_row_b, Hkv, Ls, Lr, Sc, max_seqs;
  const int* slot_ids; const int* seq_len; uint32_t* status;
};

// Output row r of one (sequence, KV head): which input row it copies, or -1 for the new token.
__device__ __forceinline__ int source_row(int r, int t, int Ls, int Lsr) {
  if (t < Lsr) return r == t ? -1 : r;          // window not full yet: plain scatter at t
  if (r < Ls || r >= Lsr) return r;             // sinks and selected rows
  return r == Lsr - 1 ? -1 : r + 1;             // window shifted by one, new token last
}

__global__ void __launch_bounds__(NT) concat_update_kernel(const ConcatArgs a) {
  const int i = blockIdx.z, h = blockIdx.y, r0 = blockIdx.x * ROWS;
  const int slot = a.slot_ids[i];
  if (slot < 0 || slot >= a.max_seqs) {
    if (threadIdx.x == 0 && blockIdx.x == 0 && h == 0 && a.status) atomicOr(a.status, SNAP_DEV_BAD_SLOT);
    return;
  }
  const int t = a.seq_len[slot], Lsr = a.Ls + a.Lr;
  const int kc = a.k_row_b / 16, vc = a.vout ? a.v_row_b / 16 : 0;
  const int nrows = min(ROWS, a.Sc - r0);
  const char* kin = a.kin + slot * a.k_seq_b + h * a.k_head_b;
  char* kout = a.kout + slot * a.k_seq_b + h * a.k_head_b;
  const char* vin = a.vin ? a.vin + slot * a.v_seq_b + h * a.v_head_b : nullptr;
  char* vout = a.vout ? a.vout + slot * a.v_seq_b + h * a.v_head_b : nullptr;
  const char* kn = a.k_new + ((long long)i * a.Hkv + h) * a.k_row_b;
  const char* vn = a.v_new ? a.v_new + ((long long)i * a.Hkv + h) * a.v_row_b : nullptr;
  for (int item = threadIdx.x; item < nrows * kc; item += NT) {
    const int r = r0 + item / kc, c = item % kc;
    const int src = source_row(r, t, a.Ls, Lsr);
    const uint4 val = src < 0 ? reinterpret_cast<const uint4*>(kn)[c]
                              : reinterpret_cast<const uint4*>(kin + (long long)src * a.k_row_b)[c];
    reinterpret_cast<uint4*>(kout + (long long)r * a.k_row_b)[c] = val;
  }
  for (int item = threadIdx.x; item < nrows * vc; item += NT) {
    const int r = r0 + item / vc, c = item % vc;
    const int src = source_row(r, t, a.Ls, Lsr);
    const uint4 val = src < 0 ? reinterpret_cast<const uint4*>(vn)[c]
                              : reinterpret_cast<const uint4*>(vin + (long long)src * a.v_row_b)[c];
    reinterpret_cast<uint4*>(vout + (long long)r * a.v_row_b)[c] = val;
  }
}

// Runs after every block of the update has read the lengths.
__global__ void bump_len_kernel(const int* slot_ids, int n_active, int* seq_len, int max_seqs) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_active) return;
  const int slot = slot_ids[i];
  if (slot >= 0 && slot < max_seqs) seq_len[slot] += 1;
}

}  // namespace
}  // namespace snap

using namespace snap;

extern "C" int snap_append_kv_concat(const snap_config_t* cfg, const snap_layout_t* layout,
                                     const void* k_new_dev, const void* v_new_dev,
                                     const int32_t* slot_ids_dev, int32_t n_active,
                                     const void* k_cache_in_dev, const void* v_cache_in_dev,
                                     void* k_cache_out_dev, void* v_cache_out_dev,
                                     int32_t* seq_len_dev, uint32_t* status_dev, void* cuda_stream) {
  snap_layout_t lay;
  const int rc = snap_cache_layout(cfg, &lay);
  if (rc != SNAP_OK) return rc;
  if (!layout) return SNAP_ERR_NULL_POINTER;
  if (n_active < 0 || layout->slots != lay.slots) return SNAP_ERR_INVALID_ARG;
  if (n_active == 0) return SNAP_OK;
  if (!k_new_dev || !slot_ids_dev || !k_cache_in_dev || !k_cache_out_dev || !seq_len_dev)
    return SNAP_ERR_NULL_POINTER;
  if (!cfg->v_aliases_k && (!v_new_dev || !v_cache_in_dev || !v_cache_out_dev)) return SNAP_ERR_NULL_POINTER;
  if (k_cache_in_dev == k_cache_out_dev || (!cfg->v_aliases_k && v_cache_in_dev == v_cache_out_dev))
    return SNAP_ERR_INVALID_ARG;                 // the update is out of place

  const int eb = cfg->dtype == SNAP_F32 ? 4 : 2;
  ConcatArgs a;
  a.k_new = static_cast<const char*>(k_new_dev);
  a.kin = static_cast<const char*>(k_cache_in_dev);
  a.kout = static_cast<char*>(k_cache_out_dev);
  if (cfg->v_aliases_k) {
    a.v_new = nullptr; a.vin = nullptr; a.vout = nullptr;
  } else {
    a.v_new = static_cast<const char*>(v_new_dev);
    a.vin = static_cast<const char*>(v_cache_in_dev);
    a.vout = static_cast<char*>(v_cache_out_dev);
  }
  a.k_row_b = cfg->d_qk * eb; a.v_row_b = cfg->d_v * eb;
  a.Hkv = cfg->n_kv_heads; a.Ls = cfg->l_sink; a.Lr = cfg->l_recent; a.Sc = lay.slots;
  a.max_seqs = cfg->max_seqs;
  a.k_head_b = (long long)a.Sc * a.k_row_b; a.k_seq_b = a.k_head_b * a.Hkv;
  a.v_head_b = (long long)a.Sc * a.v_row_b; a.v_seq_b = a.v_head_b * a.Hkv;
  a.slot_ids = slot_ids_dev; a.seq_len = seq_len_dev; a.status = status_dev;

  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  dim3 grid((a.Sc + ROWS - 1) / ROWS, a.Hkv, n_active);
  concat_update_kernel<<<grid, NT, 0, st>>>(a);
  count_launch();
  bump_len_kernel<<<(n_active + 127) / 128, 128, 0, st>>>(slot_ids_dev, n_active, seq_len_dev, cfg->max_seqs);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SNAP_OK : SNAP_ERR_CUDA;
}
