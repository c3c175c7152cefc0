// Decode attention over the compressed cache (Section 3.3), portable version: any element
// type, any head sizes, any group size (used for fp32, for latent attention until its
// tensor-core version applies, and as the fallback).
//
// Split-K flash decoding: grid = (splits, KV head x head block, sequence).  Each CTA walks
// its share of the valid slots -- [0, min(len, Lsr)) and [Lsr, Lsr + valid_topk) -- in tiles
// of 32 rows: warps compute q.k for up to 8 heads of the group, one warp per head updates the
// running max / sum (online softmax), then every thread accumulates p.V for its output
// dimensions.  Partial (m, l, acc) go to scratch and a second kernel merges the splits.
//
// Fused append (Eq. 3): when a new token is given, every CTA that meets the slot it is
// written to reads the new row instead of the stale one, and the CTA of head block 0 that
// owns the slot stores it; the sequence length is advanced by the merge kernel, after every
// split has read it.
#include "snap_internal.cuh"

namespace snap {
namespace {

constexpr int NT = 256, NWARP = NT / 32, HB = 8, TR = 32, MAX_DV_PER_THREAD = 2;

struct DecodeArgs {
  const void* q; const void* k_new; const void* v_new;
  const int* slot_ids; int n_active;
  char* kc; char* vc;
  long long kc_seq_b, kc_head_b, vc_seq_b, vc_head_b;
  int k_row_b, v_row_b;
  int Hq, Hkv, g, d_qk, d_v, Ls, Lr, max_seqs, v_aliases_k, n_hb, nsplit;
  float scale;
  int* seq_len; const int* valid_topk;
  float* partials;       // [n_active][Hq][nsplit][d_v + 2]
  void* out;
  uint32_t* status;
};

template <typename T>
__global__ void __launch_bounds__(NT) decode_split_kernel(const DecodeArgs a) {
  pdl_wait();                                // the previous step's merge (or whatever came before) has finished
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the merge may take its place and wait
  extern __shared__ float smem[];
  float* qs = smem;                          // [HB][d_qk]
  float* sc = qs + HB * a.d_qk;              // [HB][TR]
  float* m_run = sc + HB * TR;               // [HB]
  float* l_run = m_run + HB;
  float* alpha = l_run + HB;
  float* sc_x = alpha + HB;                  // [HB][NT / 2] exchange between the CTA's halves (narrow heads)

  const int sp = blockIdx.x, i = blockIdx.z;
  const int kvh = blockIdx.y / a.n_hb, hb = blockIdx.y % a.n_hb;
  const int h0 = kvh * a.g + hb * HB;                       // first query head of this block
  const int nh = min(HB, a.g - hb * HB);
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int slot = a.slot_ids[i];
  const int ps = a.d_v + 2;
  float* part = a.partials + (((long long)i * a.Hq + h0) * a.nsplit + sp) * ps;

  float acc[HB][MAX_DV_PER_THREAD];
#pragma unroll
  for (int h = 0; h < HB; ++h)
#pragma unroll
    for (int c = 0; c < MAX_DV_PER_THREAD; ++c) acc[h][c] = 0.f;

  const bool bad = slot < 0 || slot >= a.max_seqs;
  int n_low = 0, n_valid = 0, new_slot = -1;
  if (!bad) {
    const int t = a.seq_len[slot];
    const int len = t + (a.k_new ? 1 : 0);
    n_low = min(len, a.Ls + a.Lr);
    n_valid = n_low + a.valid_topk[slot];
    if (a.k_new) new_slot = ring_slot(t, a.Ls, a.Lr);
  } else if (tid == 0 && a.status) {
    atomicOr(a.status, SNAP_DEV_BAD_SLOT);
  }
  const int ntiles = (n_valid + TR - 1) / TR;
  const int tps = (ntiles + a.nsplit - 1) / a.nsplit;
  const int v0 = min(n_valid, sp * tps * TR), v1 = min(n_valid, (sp + 1) * tps * TR);

  // p.V: a thread owns output dims; with heads of at most NT / 2 dims the CTA's two halves share the rows of a
  // tile between them (their sums meet in shared memory at the end) instead of leaving one half idle
  const int nhalf = a.d_v <= NT / 2 ? 2 : 1;
  const int rhalf = nhalf == 2 ? tid / (NT / 2) : 0, dtid = nhalf == 2 ? tid % (NT / 2) : tid;
  for (int e = tid; e < nh * a.d_qk; e += NT)
    qs[e] = to_f32<T>(static_cast<const T*>(a.q)[((long long)i * a.Hq + h0) * a.d_qk + e]);
  if (tid < HB) { m_run[tid] = -INFINITY; l_run[tid] = 0.f; alpha[tid] = 1.f; }
  __syncthreads();

  const char* kc = a.kc + slot * a.kc_seq_b + kvh * a.kc_head_b;
  const char* vc = a.v_aliases_k ? kc : a.vc + slot * a.vc_seq_b + kvh * a.vc_head_b;
  const int v_row_b = a.v_aliases_k ? a.k_row_b : a.v_row_b;
  const T* kn = a.k_new ? static_cast<const T*>(a.k_new) + ((long long)i * a.Hkv + kvh) * a.d_qk : nullptr;
  const T* vn = a.v_aliases_k ? kn
                : (a.v_new ? static_cast<const T*>(a.v_new) + ((long long)i * a.Hkv + kvh) * a.d_v : nullptr);
  const int Lsr = a.Ls + a.Lr;

  constexpr int RPW = TR / NWARP;                            // rows per warp and tile
  for (int vb = v0; vb < v1; vb += TR) {
    // phase 1: logits.  A warp takes its RPW rows together, so that the loads of all of them are in flight at
    // once (row after row, each row's load latency was paid in turn: 37 us per step of a 772-slot fp32 cache).
    {
      const T* krow[RPW];
      bool live[RPW];
#pragma unroll
      for (int rr = 0; rr < RPW; ++rr) {
        const int v = vb + wid + rr * NWARP;
        live[rr] = v < v1;
        const int cs = v < n_low ? v : Lsr + (v - n_low);
        krow[rr] = !live[rr] ? nullptr : cs == new_slot ? kn : reinterpret_cast<const T*>(kc + (long long)cs * a.k_row_b);
      }
      float s[RPW][HB];
#pragma unroll
      for (int rr = 0; rr < RPW; ++rr)
#pragma unroll
        for (int h = 0; h < HB; ++h) s[rr][h] = 0.f;
#pragma unroll 2
      for (int c = lane; c < a.d_qk; c += 32) {
        float kv[RPW];
#pragma unroll
        for (int rr = 0; rr < RPW; ++rr) kv[rr] = live[rr] ? to_f32<T>(krow[rr][c]) : 0.f;
#pragma unroll
        for (int h = 0; h < HB; ++h) {
          if (h < nh) {
            const float qv = qs[h * a.d_qk + c];
#pragma unroll
            for (int rr = 0; rr < RPW; ++rr) s[rr][h] = fmaf(kv[rr], qv, s[rr][h]);
          }
        }
      }
#pragma unroll
      for (int rr = 0; rr < RPW; ++rr) {
#pragma unroll
        for (int h = 0; h < HB; ++h) {
          if (h < nh) {                                      // nh is uniform over the CTA
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s[rr][h] += __shfl_xor_sync(0xffffffffu, s[rr][h], o);
          }
        }
        if (lane == 0) {
          const int r = wid + rr * NWARP;
#pragma unroll
          for (int h = 0; h < HB; ++h) sc[h * TR + r] = live[rr] ? s[rr][h] * a.scale : -INFINITY;
        }
      }
    }
    __syncthreads();
    // phase 2: online softmax, one warp per head
    if (wid < nh) {
      const float s = sc[wid * TR + lane];
      float tmax = s;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
      const float m_old = m_run[wid];
      const float m_new = fmaxf(m_old, tmax);
      const float p = s == -INFINITY ? 0.f : expf(s - m_new);
      float sum = p;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      sc[wid * TR + lane] = p;
      if (lane == 0) {
        const float al = m_old == -INFINITY ? 0.f : expf(m_old - m_new);
        alpha[wid] = al;
        l_run[wid] = l_run[wid] * al + sum;
        m_run[wid] = m_new;
      }
    }
    __syncthreads();
    // phase 3: accumulate p.V
#pragma unroll
    for (int h = 0; h < HB; ++h) {
      if (h < nh) {
        const float al = alpha[h];
#pragma unroll
        for (int c = 0; c < MAX_DV_PER_THREAD; ++c) acc[h][c] *= al;
      }
    }
    const int nr = min(TR, v1 - vb);
    constexpr int VB = 8;                                    // value rows whose loads are in flight together
    for (int r0 = rhalf * VB; r0 < nr; r0 += VB * nhalf) {   // narrow heads: the two halves of the CTA take alternate groups
#pragma unroll
      for (int c = 0; c < MAX_DV_PER_THREAD; ++c) {
        const int dim = dtid + c * NT;
        if (dim < a.d_v) {
          float vv[VB];
#pragma unroll
          for (int u = 0; u < VB; ++u) {
            const int v = vb + r0 + u;
            const int cs = v < n_low ? v : Lsr + (v - n_low);
            const T* vrow = cs == new_slot ? vn : reinterpret_cast<const T*>(vc + (long long)cs * v_row_b);
            vv[u] = r0 + u < nr ? to_f32<T>(vrow[dim]) : 0.f;
          }
#pragma unroll
          for (int u = 0; u < VB; ++u) {
#pragma unroll
            for (int h = 0; h < HB; ++h)
              if (h < nh) acc[h][c] = fmaf(sc[h * TR + r0 + u], vv[u], acc[h][c]);
          }
        }
      }
    }
    __syncthreads();
  }

  // partial results
  if (nhalf == 2) {
    float* xs = sc_x;
    if (rhalf == 1) {
#pragma unroll
      for (int h = 0; h < HB; ++h) xs[h * (NT / 2) + dtid] = acc[h][0];
    }
    __syncthreads();
    if (rhalf == 0) {
#pragma unroll
      for (int h = 0; h < HB; ++h) acc[h][0] += xs[h * (NT / 2) + dtid];
    }
  }
#pragma unroll
  for (int h = 0; h < HB; ++h) {
    if (h < nh) {
      float* ph = part + (long long)h * a.nsplit * ps;
      if (tid == 0) { ph[0] = m_run[h]; ph[1] = l_run[h]; }
#pragma unroll
      for (int c = 0; c < MAX_DV_PER_THREAD; ++c) {
        const int dim = dtid + c * NT;
        if (rhalf == 0 && dim < a.d_v) ph[2 + dim] = acc[h][c];
      }
    }
  }

  // the CTA that owns the new token's slot stores it (head block 0 only)
  if (new_slot >= 0 && hb == 0 && new_slot >= v0 && new_slot < v1) {
    const int kvec = a.k_row_b / 16;
    char* dstk = a.kc + slot * a.kc_seq_b + kvh * a.kc_head_b + (long long)new_slot * a.k_row_b;
    for (int c = tid; c < kvec; c += NT)
      reinterpret_cast<uint4*>(dstk)[c] = reinterpret_cast<const uint4*>(kn)[c];
    if (!a.v_aliases_k) {
      const int vvec = a.v_row_b / 16;
      char* dstv = a.vc + slot * a.vc_seq_b + kvh * a.vc_head_b + (long long)new_slot * a.v_row_b;
      for (int c = tid; c < vvec; c += NT)
        reinterpret_cast<uint4*>(dstv)[c] = reinterpret_cast<const uint4*>(vn)[c];
    }
  }
}

// Merge the splits of one (sequence, query head): out = sum_s acc_s e^{m_s - m} / sum_s l_s e^{m_s - m}.
template <typename T>
__global__ void decode_merge_kernel(const float* __restrict__ partials, T* __restrict__ out,
                                    int Hq, int d_v, int nsplit, const int* __restrict__ slot_ids,
                                    int* seq_len, int max_seqs, int bump) {
  pdl_wait();                                // all splits have written their partial results
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next step's kernel waits at its top
  const int h = blockIdx.x, i = blockIdx.y;
  const int ps = d_v + 2;
  const float* p = partials + ((long long)i * Hq + h) * nsplit * ps;
  // The splits' (m, l) are fetched by one thread each and their weights e^{m_s - m} computed once per block;
  // the sums over the splits then run with eight loads in flight.  (One load after the other, per thread and
  // per split, this kernel took 12.5 us for 13 splits of 8 heads.)
  __shared__ float m_s[64], w_s[64], wl_s[64];               // nsplit <= 64
  const int tid = threadIdx.x;
  float l_mine = 0.f;
  if (tid < nsplit) {
    m_s[tid] = p[tid * ps];
    l_mine = p[tid * ps + 1];
  }
  __syncthreads();
  float m = -INFINITY;
  for (int s = 0; s < nsplit; ++s) m = fmaxf(m, m_s[s]);
  if (tid < nsplit) {
    const float w = m_s[tid] != -INFINITY ? expf(m_s[tid] - m) : 0.f;
    w_s[tid] = w;
    wl_s[tid] = w * l_mine;
  }
  __syncthreads();
  float l = 0.f;
  for (int s = 0; s < nsplit; ++s) l += wl_s[s];             // same order in every thread
  const float inv = l > 0.f ? 1.f / l : 0.f;
  for (int dim = tid; dim < d_v; dim += blockDim.x) {
    float o = 0.f;
#pragma unroll 8
    for (int s = 0; s < nsplit; ++s) o = fmaf(w_s[s], p[s * ps + 2 + dim], o);
    out[((long long)i * Hq + h) * d_v + dim] = from_f32<T>(o * inv);
  }
  if (bump && h == 0 && threadIdx.x == 0) {
    const int slot = slot_ids[i];
    if (slot >= 0 && slot < max_seqs) seq_len[slot] += 1;
  }
}

}  // namespace

int decode_generic_nsplit(const Shape& s, int n_active, int sm_count) {
  const int n_hb = (s.g + HB - 1) / HB;
  const long long base = (long long)n_active * s.Hkv * n_hb;
  int nsplit = (int)((4LL * sm_count + base - 1) / base);
  const int max_split = (s.Sc + TR - 1) / TR;               // down to one 32-row tile per CTA
  nsplit = nsplit < 1 ? 1 : nsplit;
  nsplit = nsplit > max_split ? max_split : nsplit;
  nsplit = nsplit > 64 ? 64 : nsplit;
  return nsplit < 1 ? 1 : nsplit;
}

size_t decode_partial_floats(const Shape& s, int n_active, int nsplit) {
  return (size_t)n_active * s.Hq * nsplit * (s.d_v + 2);
}

cudaError_t launch_decode_generic(int dtype, const Shape& s, const void* q, const void* k_new,
                                  const void* v_new, const int* slot_ids, int n_active,
                                  void* k_cache, void* v_cache, int* seq_len,
                                  const int* valid_topk, void* out, float* partials, int nsplit,
                                  uint32_t* status, cudaStream_t st) {
  if (n_active == 0) return cudaSuccess;
  const int eb = dtype == SNAP_F32 ? 4 : 2;
  DecodeArgs a;
  a.q = q; a.k_new = k_new; a.v_new = v_new; a.slot_ids = slot_ids; a.n_active = n_active;
  a.kc = static_cast<char*>(k_cache); a.vc = static_cast<char*>(v_cache);
  a.k_row_b = s.d_qk * eb; a.v_row_b = s.d_v * eb;
  a.kc_head_b = (long long)s.Sc * a.k_row_b; a.kc_seq_b = a.kc_head_b * s.Hkv;
  a.vc_head_b = (long long)s.Sc * a.v_row_b; a.vc_seq_b = a.vc_head_b * s.Hkv;
  a.Hq = s.Hq; a.Hkv = s.Hkv; a.g = s.g; a.d_qk = s.d_qk; a.d_v = s.d_v; a.Ls = s.Ls; a.Lr = s.Lr;
  a.max_seqs = s.max_seqs; a.v_aliases_k = s.v_aliases_k; a.n_hb = (s.g + HB - 1) / HB;
  a.nsplit = nsplit; a.scale = s.scale; a.seq_len = seq_len; a.valid_topk = valid_topk;
  a.partials = partials; a.out = out; a.status = status;
  const size_t smem = (size_t)(HB * s.d_qk + HB * TR + 3 * HB + HB * (NT / 2)) * sizeof(float);
  dim3 grid(nsplit, s.Hkv * a.n_hb, n_active);
  dim3 mgrid(s.Hq, n_active);
  const int bump = k_new != nullptr;
  // both launches are programmatic dependents: each waits at its top for the one before
  cudaError_t e;
  if (dtype == SNAP_F32) {
    e = launch_pdl(decode_split_kernel<float>, grid, dim3(NT), smem, st, a);
    count_launch();
    if (e == cudaSuccess)
      e = launch_pdl(decode_merge_kernel<float>, mgrid, dim3(128), 0, st, static_cast<const float*>(partials),
                     static_cast<float*>(out), s.Hq, s.d_v, nsplit, slot_ids, seq_len, s.max_seqs, bump);
  } else {
    e = launch_pdl(decode_split_kernel<__nv_bfloat16>, grid, dim3(NT), smem, st, a);
    count_launch();
    if (e == cudaSuccess)
      e = launch_pdl(decode_merge_kernel<__nv_bfloat16>, mgrid, dim3(128), 0, st, static_cast<const float*>(partials),
                     static_cast<__nv_bfloat16*>(out), s.Hq, s.d_v, nsplit, slot_ids, seq_len, s.max_seqs, bump);
  }
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace snap
