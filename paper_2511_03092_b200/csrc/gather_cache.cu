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
#include <cstring>

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
  int* idx;
  int* seq_len; int* valid_topk;
  uint32_t* status;
  // the verdict of the double-precision re-scoring of the selection (head == NULL: there was none)
  RefineBuffers ref;
  float* P; int c_stride;                              // pooled-score scratch, free by now: holds the old index list
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
                                          const int* __restrict__ idx_row, uint32_t* status) {
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
        if (p >= 0 && index_ok(p, L, status)) val[u] = __ldg(reinterpret_cast<const uint4*>(src_base + (long long)p * tok_b) + chunk_of[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (slot_of[u] >= 0) reinterpret_cast<uint4*>(dst_base + (long long)slot_of[u] * row_b)[chunk_of[u]] = val[u];
  }
}

// The re-scoring found that n positions leave the selection of a (prompt, KV head) and n others
// enter it.  Run by the last CTA of the head, after every CTA of the head has finished copying:
// rewrite the ascending index list and copy again the cache rows of the ranks whose position changed.
struct CorrectionArgs {
  const int* leaving; const int* entering;   // candidate indices (position - Ls), n of each
  int* out; int* old;                        // the head's index list, and scratch for its previous content
  const char* ksrc; const char* vsrc; char* kdst; char* vdst;   // this head's prompt rows and cache rows (v: NULL if aliased)
  long long k_tok_b, v_tok_b;
  int k_row_b, v_row_b, n, K, Ls, Lsr, L;
  uint32_t* status;
};
__device__ __noinline__ void apply_selection_correction(const CorrectionArgs c) {
  const int tid = threadIdx.x;
  for (int i = tid; i < c.K; i += NT) c.old[i] = c.out[i];
  __syncthreads();
  auto shift_of = [&](int j) {                               // entering below j minus leaving below j
    int sft = 0;
    for (int u = 0; u < c.n; ++u) sft += (c.entering[u] < j) - (c.leaving[u] < j);
    return sft;
  };
  for (int i = tid; i < c.K; i += NT) {
    const int j = c.old[i] - c.Ls;
    bool leaves = false;
    for (int u = 0; u < c.n; ++u) leaves |= c.leaving[u] == j;
    if (!leaves && index_ok(i + shift_of(j), c.K, c.status)) c.out[i + shift_of(j)] = c.old[i];
  }
  for (int u = tid; u < c.n; u += NT) {
    const int j = c.entering[u], pos_abs = c.Ls + j;
    int lo = 0, hi = c.K;                                    // entries of the old list below this one
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (c.old[mid] < pos_abs) lo = mid + 1; else hi = mid;
    }
    if (index_ok(lo + shift_of(j), c.K, c.status)) c.out[lo + shift_of(j)] = pos_abs;
  }
  __syncthreads();
  // Copy again the rows of the ranks whose position changed (everything between a leaving and an
  // entering position moves by one rank).  Ranks are scanned 1024 at a time into a list in shared
  // memory, then all threads copy the listed rows, 16 bytes per thread and turn.
  __shared__ int changed[1024], changed_pos[1024];
  __shared__ int n_changed;
  const int kv = c.k_row_b / 16, vv = c.vdst ? c.v_row_b / 16 : 0;
  for (int base = 0; base < c.K; base += 1024) {
    if (tid == 0) n_changed = 0;
    __syncthreads();
    for (int i = base + tid; i < min(base + 1024, c.K); i += NT) {
      const int pos = c.out[i];
      if (pos != c.old[i] && index_ok(pos, c.L, c.status)) {
        const int e = atomicAdd(&n_changed, 1);
        changed[e] = i;
        changed_pos[e] = pos;
      }
    }
    __syncthreads();
    const int total = n_changed * (kv + vv);
    for (int e0 = tid; e0 < total; e0 += 4 * NT) {            // four 16-byte loads in flight per thread
      uint4 val[4];
      uint4* dst[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int e = e0 + u * NT;
        dst[u] = nullptr;
        if (e < total) {
          const int r = e / (kv + vv), v = e % (kv + vv);
          const long long pos = changed_pos[r], i = changed[r];
          if (v < kv) {
            val[u] = reinterpret_cast<const uint4*>(c.ksrc + pos * c.k_tok_b)[v];
            dst[u] = reinterpret_cast<uint4*>(c.kdst + (c.Lsr + i) * c.k_row_b) + v;
          } else {
            val[u] = reinterpret_cast<const uint4*>(c.vsrc + pos * c.v_tok_b)[v - kv];
            dst[u] = reinterpret_cast<uint4*>(c.vdst + (c.Lsr + i) * c.v_row_b) + (v - kv);
          }
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (dst[u]) *dst[u] = val[u];
    }
    __syncthreads();
  }
}

__global__ void __launch_bounds__(NT, 6) gather_kernel(const GatherArgs a) {
  // With a re-scoring kernel in front, this grid was released by that kernel after its own wait:
  // the selection kernel's index list is complete, and the re-scoring's verdict is read at the end.
  if (!a.ref.head) pdl_wait();
  const int seq = blockIdx.z, kvh = blockIdx.y;
  const int L = a.b.len[seq], slot = a.b.slot[seq];
  if (slot < 0 || slot >= a.max_seqs) {
    if (threadIdx.x == 0 && a.status) atomicOr(a.status, SNAP_DEV_BAD_SLOT);
    if (a.ref.head) pdl_wait();                              // this grid must not finish before the one in front of it
    return;
  }
  const int Lsr = a.Ls + a.Lr;
  const int vt = min(max(L - Lsr, 0), a.K);
  const int* idx_row = a.idx ? a.idx + ((long long)(a.b.first_seq + seq) * a.Hkv + kvh) * a.K : nullptr;
  const int s0 = blockIdx.x * ROWS;
  const long long tok0 = a.b.tok_off[seq];
  copy_rows(a.k + tok0 * a.k_tok_b + kvh * a.k_head_b, a.k_tok_b,
            a.kc + slot * a.kc_seq_b + kvh * a.kc_head_b, a.k_row_b, s0, a.Sc, L, a.Ls, a.Lr, vt,
            idx_row, a.status);
  if (a.vc)
    copy_rows(a.v + tok0 * a.v_tok_b + kvh * a.v_head_b, a.v_tok_b,
              a.vc + slot * a.vc_seq_b + kvh * a.vc_head_b, a.v_row_b, s0, a.Sc, L, a.Ls, a.Lr, vt,
              idx_row, a.status);
  if (blockIdx.x == 0 && kvh == 0 && threadIdx.x == 0) {
    a.seq_len[slot] = L;
    a.valid_topk[slot] = vt;
  }
  if (!a.ref.head) return;
  pdl_wait();                                                // the re-scoring kernel has finished
  const int si = a.b.score_idx[seq];
  if (si < 0) return;
  const long long z = (long long)si * a.Hkv + kvh;
  RefineHead* head = a.ref.head + z;
  const int n = head->changed;
  if (n <= 0) return;                                        // the single-precision order stands (the usual case)
  __shared__ int last_s;
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    last_s = atomicAdd(&head->gather_done, 1) == (int)gridDim.x - 1;
    __threadfence();
  }
  __syncthreads();
  if (last_s) {
    CorrectionArgs c;
    c.leaving = a.ref.lists + z * 2 * a.ref.cap; c.entering = c.leaving + a.ref.cap;
    c.out = a.idx + ((long long)(a.b.first_seq + seq) * a.Hkv + kvh) * a.K;
    c.old = reinterpret_cast<int*>(a.P + z * a.c_stride);
    c.ksrc = a.k + tok0 * a.k_tok_b + kvh * a.k_head_b;
    c.kdst = a.kc + slot * a.kc_seq_b + kvh * a.kc_head_b;
    c.vsrc = a.vc ? a.v + tok0 * a.v_tok_b + kvh * a.v_head_b : nullptr;
    c.vdst = a.vc ? a.vc + slot * a.vc_seq_b + kvh * a.vc_head_b : nullptr;
    c.k_tok_b = a.k_tok_b; c.v_tok_b = a.v_tok_b; c.k_row_b = a.k_row_b; c.v_row_b = a.v_row_b;
    c.n = n; c.K = a.K; c.Ls = a.Ls; c.Lsr = Lsr; c.L = L; c.status = a.status;
    apply_selection_correction(c);
  }
}

struct AppendArgs {
  const char* k_new; const char* v_new;
  char* kc; char* vc;
  long long kc_seq_b, kc_head_b, vc_seq_b, vc_head_b;
  int k_row_b, v_row_b, Hkv, Ls, Lr, Sc, max_seqs, n_active;
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
  if (!index_ok(dst, a.Sc, a.status) || !index_ok(t, 0x7fffffff, a.status)) return;
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
                          int* idx, void* k_cache, void* v_cache, int* seq_len,
                          int* valid_topk, uint32_t* status, cudaStream_t st, const ScoreBuffers* buf) {
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
  std::memset(&a.ref, 0, sizeof(a.ref));
  a.P = nullptr; a.c_stride = 0;
  if (buf && buf->ref.head && b.n_scored > 0 && s.K > 0) { a.ref = buf->ref; a.P = buf->P; a.c_stride = buf->c_stride; }
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
  a.Hkv = s.Hkv; a.Ls = s.Ls; a.Lr = s.Lr; a.Sc = s.Sc; a.max_seqs = s.max_seqs; a.n_active = n_active;
  a.slot_ids = slot_ids; a.seq_len = seq_len; a.status = status;
  append_kernel<<<n_active, NT, 0, st>>>(a);
  count_launch();
  return cudaGetLastError();
}

}  // namespace snap
