// Cache construction at prefill (Section 3.2.1 ring build + the top-K gather of Section 3.2.2)
// and the stand-alone Eq. 3 scatter of one new token.
//
// For every cache slot the source prompt position is computed directly:
//   slot s < Ls             -> position s                       (sinks)
//   Ls <= s < Lsr           -> the position p in [max(Ls, L-Lr), L) with (p - Ls) mod Lr == s - Ls
//                              (the two ring-aligned ranges of the paper's ring-buffer figure)
//   s >= Lsr                -> idx[s - Lsr] for the first valid_topk entries
// and rows with no source are zero-filled, so a slot is fully rewritten by one launch.
// Rows move as 16-byte vectors; a row's vectors are read and written by adjacent threads.
#include "snap_internal.cuh"

namespace snap {
namespace {

constexpr int NT = 256, ROWS = 64;

struct GatherArgs {
  const char* k; const char* v;
  long long k_tok_b, k_head_b, v_tok_b, v_head_b;      // source strides in bytes
  char* kc; char* vc;
  long long kc_seq_b, kc_head_b, vc_seq_b, vc_head_b;  // cache strides in bytes
  int k_row_b, v_row_b;
  int Hkv, Ls, Lr, K, Sc, max_seqs;
  SeqBatch b;
  const int* idx;
  int* seq_len; int* valid_topk;
  uint32_t* status;
};

__device__ __forceinline__ int source_position(int s, int L, int Ls, int Lr, int vt,
                                               const int* __restrict__ idx_row) {
  if (s < Ls) return s < L ? s : -1;
  const int Lsr = Ls + Lr;
  if (s < Lsr) {
    if (L <= Ls) return -1;
    const int r = s - Ls, q = L - 1 - Ls;
    const int off = ((q - r) % Lr + Lr) % Lr;
    const int p = L - 1 - off;
    return p >= Ls ? p : -1;
  }
  const int i = s - Lsr;
  return i < vt ? idx_row[i] : -1;
}

__device__ __forceinline__ void copy_rows(const char* __restrict__ src_base, long long tok_b,
                                          char* __restrict__ dst_base, int row_b, int s0, int Sc,
                                          int L, int Ls, int Lr, int vt,
                                          const int* __restrict__ idx_row) {
  const int vecs = row_b / 16, total = ROWS * vecs;
  // four independent 16-byte loads are in flight per thread before anything is stored
  for (int base = threadIdx.x; base < total; base += 4 * NT) {
    uint4 val[4];
    int slot_of[4], chunk_of[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int item = base + u * NT;
      const int s = s0 + item / vecs;
      slot_of[u] = item < total && s < Sc ? s : -1;
      chunk_of[u] = item % vecs;
      val[u] = make_uint4(0u, 0u, 0u, 0u);
      if (slot_of[u] >= 0) {
        const int p = source_position(s, L, Ls, Lr, vt, idx_row);
        if (p >= 0) val[u] = __ldg(reinterpret_cast<const uint4*>(src_base + (long long)p * tok_b) + chunk_of[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (slot_of[u] >= 0) reinterpret_cast<uint4*>(dst_base + (long long)slot_of[u] * row_b)[chunk_of[u]] = val[u];
  }
}

__global__ void __launch_bounds__(NT) gather_kernel(const GatherArgs a) {
  pdl_wait();
  // the refinement of the selection (launched next) may start now: it reads only what the selection
  // kernel wrote, and waits for this grid itself before it corrects anything
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int seq = blockIdx.z, kvh = blockIdx.y;
  const int L = a.b.len[seq], slot = a.b.slot[seq];
  if (slot < 0 || slot >= a.max_seqs) {
    if (threadIdx.x == 0 && a.status) atomicOr(a.status, SNAP_DEV_BAD_SLOT);
    return;
  }
  const int Lsr = a.Ls + a.Lr;
  const int vt = min(max(L - Lsr, 0), a.K);
  const int* idx_row = a.idx ? a.idx + ((long long)(a.b.first_seq + seq) * a.Hkv + kvh) * a.K : nullptr;
  const int s0 = blockIdx.x * ROWS;
  const long long tok0 = a.b.tok_off[seq];
  copy_rows(a.k + tok0 * a.k_tok_b + kvh * a.k_head_b, a.k_tok_b,
            a.kc + slot * a.kc_seq_b + kvh * a.kc_head_b, a.k_row_b, s0, a.Sc, L, a.Ls, a.Lr, vt,
            idx_row);
  if (a.vc)
    copy_rows(a.v + tok0 * a.v_tok_b + kvh * a.v_head_b, a.v_tok_b,
              a.vc + slot * a.vc_seq_b + kvh * a.vc_head_b, a.v_row_b, s0, a.Sc, L, a.Ls, a.Lr, vt,
              idx_row);
  if (blockIdx.x == 0 && kvh == 0 && threadIdx.x == 0) {
    a.seq_len[slot] = L;
    a.valid_topk[slot] = vt;
  }
}

struct AppendArgs {
  const char* k_new; const char* v_new;
  char* kc; char* vc;
  long long kc_seq_b, kc_head_b, vc_seq_b, vc_head_b;
  int k_row_b, v_row_b, Hkv, Ls, Lr, max_seqs, n_active;
  const int* slot_ids; int* seq_len; uint32_t* status;
};

// One CTA per sequence: every thread reads the length before the barrier, thread 0 bumps it after.
__global__ void __launch_bounds__(NT) append_kernel(const AppendArgs a) {
  const int i = blockIdx.x;
  const int slot = a.slot_ids[i];
  if (slot < 0 || slot >= a.max_seqs) {
    if (threadIdx.x == 0 && a.status) atomicOr(a.status, SNAP_DEV_BAD_SLOT);
    return;
  }
  const int t = a.seq_len[slot];
  __syncthreads();
  const int dst = ring_slot(t, a.Ls, a.Lr);
  const int kv = a.k_row_b / 16, vv = a.vc ? a.v_row_b / 16 : 0;
  for (int item = threadIdx.x; item < a.Hkv * (kv + vv); item += NT) {
    const int h = item / (kv + vv), c = item % (kv + vv);
    if (c < kv) {
      const uint4 val = reinterpret_cast<const uint4*>(a.k_new + ((long long)i * a.Hkv + h) * a.k_row_b)[c];
      reinterpret_cast<uint4*>(a.kc + slot * a.kc_seq_b + h * a.kc_head_b + (long long)dst * a.k_row_b)[c] = val;
    } else {
      const uint4 val = reinterpret_cast<const uint4*>(a.v_new + ((long long)i * a.Hkv + h) * a.v_row_b)[c - kv];
      reinterpret_cast<uint4*>(a.vc + slot * a.vc_seq_b + h * a.vc_head_b + (long long)dst * a.v_row_b)[c - kv] = val;
    }
  }
  if (threadIdx.x == 0) a.seq_len[slot] = t + 1;
}

inline int elt_bytes(int dtype) { return dtype == SNAP_F32 ? 4 : 2; }

}  // namespace

cudaError_t launch_gather(int dtype, const Shape& s, const SeqBatch& b, const KVSource& src,
                          const int* idx, void* k_cache, void* v_cache, int* seq_len,
                          int* valid_topk, uint32_t* status, cudaStream_t st) {
  if (b.n == 0) return cudaSuccess;
  const int eb = elt_bytes(dtype);
  GatherArgs a;
  a.k = static_cast<const char*>(src.k); a.v = static_cast<const char*>(src.v);
  a.k_tok_b = src.k_tok_stride * eb; a.k_head_b = src.k_head_stride * eb;
  a.v_tok_b = src.v_tok_stride * eb; a.v_head_b = src.v_head_stride * eb;
  a.kc = static_cast<char*>(k_cache);
  a.vc = s.v_aliases_k ? nullptr : static_cast<char*>(v_cache);
  a.k_row_b = s.d_qk * eb; a.v_row_b = s.d_v * eb;
  a.kc_head_b = (long long)s.Sc * a.k_row_b; a.kc_seq_b = a.kc_head_b * s.Hkv;
  a.vc_head_b = (long long)s.Sc * a.v_row_b; a.vc_seq_b = a.vc_head_b * s.Hkv;
  a.Hkv = s.Hkv; a.Ls = s.Ls; a.Lr = s.Lr; a.K = s.K; a.Sc = s.Sc; a.max_seqs = s.max_seqs;
  a.b = b; a.idx = s.K > 0 ? idx : nullptr;
  a.seq_len = seq_len; a.valid_topk = valid_topk; a.status = status;
  dim3 grid((s.Sc + ROWS - 1) / ROWS, s.Hkv, b.n);
  const cudaError_t e = launch_pdl(gather_kernel, grid, dim3(NT), 0, st, a);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_append(int dtype, const Shape& s, const void* k_new, const void* v_new,
                          const int* slot_ids, int n_active, void* k_cache, void* v_cache,
                          int* seq_len, uint32_t* status, cudaStream_t st) {
  if (n_active == 0) return cudaSuccess;
  const int eb = elt_bytes(dtype);
  AppendArgs a;
  a.k_new = static_cast<const char*>(k_new); a.v_new = static_cast<const char*>(v_new);
  a.kc = static_cast<char*>(k_cache);
  a.vc = s.v_aliases_k ? nullptr : static_cast<char*>(v_cache);
  a.k_row_b = s.d_qk * eb; a.v_row_b = s.d_v * eb;
  a.kc_head_b = (long long)s.Sc * a.k_row_b; a.kc_seq_b = a.kc_head_b * s.Hkv;
  a.vc_head_b = (long long)s.Sc * a.v_row_b; a.vc_seq_b = a.vc_head_b * s.Hkv;
  a.Hkv = s.Hkv; a.Ls = s.Ls; a.Lr = s.Lr; a.max_seqs = s.max_seqs; a.n_active = n_active;
  a.slot_ids = slot_ids; a.seq_len = seq_len; a.status = status;
  append_kernel<<<n_active, NT, 0, st>>>(a);
  count_launch();
  return cudaGetLastError();
}

}  // namespace snap
