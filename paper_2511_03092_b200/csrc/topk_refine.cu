// Exact selection at the top-K threshold (Eq. 2): double-precision re-scoring of the band.
//
// The score kernels compute Eq. 4 / Eq. 1 in single precision (bf16 products are exact in fp32,
// but the accumulation and the hardware exponential leave a relative error of a few 1e-7 on a
// pooled score).  Two candidates whose pooled scores lie closer together than that can come out
// in the wrong order, and at the K-th place that exchanges a selected index for a rejected one.
// The selection kernel therefore lists the band -- every candidate whose single-precision
// pooled score is within a relative distance `rel` (far larger than that error) of the K-th
// largest -- and counts the candidates above it.  Here the band members' pooled scores are
// recomputed from the inputs in double precision:
//
//   C[j'] = sum over the KV head's g * Lo window rows i of 2^(log2(e) * scale * q_i . k_j' - mu_i)
//   P[j]  = pool_w(C)[j]      (w taps around j, zero / -inf padding as in the selection kernel)
//
// with mu_i the log2-domain normaliser of Eq. 4 from the first score pass (its value as the
// statistics merge computed it in double where that is available).  The K - n_sure best band
// members by (P descending, index ascending) are the selected ones.  Where that differs from
// the single-precision choice, the positions that leave and enter the selection are handed to
// the gather kernel, which rewrites the index list and copies the affected cache rows again.
//
// The kernel runs between the selection and the gather kernel and releases the gather at once
// (the gather copies with the single-precision list and looks at the verdict when it is done),
// so the re-scoring overlaps the gather.
//
// Work split: one item = one band member x one block of 64 window rows.  The dot products are a
// small double-precision matrix product -- 64 rows x d columns against the member's w key rows
// (taps) -- on the FP64 tensor-core instruction mma.m8n8k4: a warp owns 8 rows, the taps are
// the 8 columns of the product; queries and keys are converted to double on their way into
// shared memory.  CTAs of a head stride over its items; per-item column sums go to scratch and
// the last CTA of the head to finish (a counter, no waiting) adds them in a fixed order and
// ranks the band, so the result does not depend on the order in which CTAs ran.  A band larger than its buffer is left in single-precision order and
// SNAP_DEV_BAND_OVERFLOW is raised.
#include "snap_internal.cuh"

namespace snap {
namespace {

constexpr int NT = 256;      // threads per CTA
constexpr int RB = 64;       // window rows per item (8 per warp)
constexpr int TG = 8;        // taps per pass = columns of the m8n8k4 product
constexpr int QTILE_B = 76 * 1024;   // shared memory for the staged query rows (two CTAs per SM with the key rows beside it)
constexpr int MAXCAP = 512;  // band members the ranking step holds in shared memory

struct RefineArgs {
  const void* q;            // [prompts][Hq][Lo][d]
  KVSource src;             // prompt keys / values (strides in elements)
  int Hq, Hkv, g, Lo, d, Ls, Lr, K, w, pool_mode, R, elt;
  int dc;                   // query columns staged at a time (a multiple of 16)
  double scale_log2;
  SeqBatch b;
  ScoreBuffers buf;
  uint32_t* status;
};

// two consecutive elements -> two floats (exact for both element types)
template <typename T> struct Pair;
template <> struct Pair<float> {
  using raw = float2;
  static __device__ __forceinline__ float2 to_f32(float2 v) { return v; }
};
template <> struct Pair<__nv_bfloat16> {
  using raw = uint32_t;
  static __device__ __forceinline__ float2 to_f32(uint32_t v) {
    return make_float2(__uint_as_float(v << 16), __uint_as_float(v & 0xffff0000u));
  }
};
__device__ __forceinline__ double elem_f64(const float* p) { return (double)*p; }
__device__ __forceinline__ double elem_f64(const __nv_bfloat16* p) {
  return (double)__uint_as_float((uint32_t)*reinterpret_cast<const unsigned short*>(p) << 16);
}

__device__ __forceinline__ void dmma(double& c0, double& c1, double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
               : "+d"(c0), "+d"(c1) : "d"(a), "d"(b));
}

template <typename T>
__global__ void __launch_bounds__(NT, 2) topk_refine_kernel(const RefineArgs a) {
  pdl_wait();                                               // the selection kernel has written band and counters
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the gather may start: it needs nothing from here yet
  extern __shared__ __align__(16) float smem_f[];           // [TG][d + 4] key rows as floats (exact), then [RB] query rows as loaded
  __shared__ double red[NT / 32][TG];
  __shared__ double p64[MAXCAP];
  __shared__ int jidx[MAXCAP];                              // candidate index of each band member
  __shared__ int lists[2][MAXCAP];                          // indices leaving / entering the selection
  __shared__ int n_list[2];
  __shared__ float dev_s[NT / 32];
  __shared__ int last_s;
  using raw_t = typename Pair<T>::raw;

  const int z = blockIdx.y, si = z / a.Hkv, kvh = z % a.Hkv;
  const int seq = a.b.seq_of_score[si];
  const int Le = a.b.len[seq] - a.Ls - a.Lr;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const RefineBuffers& rf = a.buf.ref;
  RefineHead* head = rf.head + z;
  const BandEntry* band = rf.band + (long long)z * rf.cap;
  const int nb_raw = head->n_band;
  const bool overflow = nb_raw > rf.cap || nb_raw > MAXCAP;
  const int nb = overflow ? 0 : nb_raw;
  const int chunks = rf.chunks, r = a.w / 2, d = a.d, KS = d + 4;
  float* ksf = smem_f;
  char* qt = reinterpret_cast<char*>(smem_f + TG * KS);
  const int q_pitch = a.dc * (int)sizeof(T) + 16;             // bytes per staged row: 4 words mod 8, conflict-free fragment loads
  double* part = rf.part + (long long)z * rf.cap * chunks * a.w;

  const T* qbase = static_cast<const T*>(a.q) + ((long long)(a.b.first_seq + seq) * a.Hq + (long long)kvh * a.g) * a.Lo * d;
  const T* kbase = static_cast<const T*>(a.src.k) + (long long)(a.b.tok_off[seq] + a.Ls) * a.src.k_tok_stride +
                   (long long)kvh * a.src.k_head_stride;
  const int frow = lane >> 2, fk = lane & 3;                 // fragment coordinates of m8n8k4

  // A CTA takes a contiguous run of items, ordered row block first: while the row block stays the
  // same (and a whole row fits the tile) the staged query rows are reused from member to member.
  const int n_items = nb * chunks, per_cta = (n_items + (int)gridDim.x - 1) / (int)gridDim.x;
  const int item_end = min(n_items, ((int)blockIdx.x + 1) * per_cta);
  int staged_chunk = -1;
  for (int item = blockIdx.x * per_cta; item < item_end; ++item) {
    const int c = item / nb, m = item - c * nb;
    const int j = band[m].idx_flag & 0x7fffffff;
    if (!index_ok(j, Le, a.status)) continue;                // uniform over the CTA
    const int row0 = c * RB, row = row0 + wid * 8 + frow;    // this item's first window row; this lane's row
    double mu = 0.0;
    if (row < a.R) {
      if (a.buf.ext_mu) {
        mu = (double)a.buf.ext_mu[((long long)(a.b.first_seq + seq) * a.Hq + (long long)kvh * a.g) * a.Lo + row];
      } else if (rf.mu64) {
        mu = rf.mu64[(long long)z * a.R + row];
      } else {
        const float2 st = a.buf.stats[(long long)z * a.R + row];
        mu = rf.stats_natural ? ((double)st.x - log((double)st.y)) * 1.4426950408889634074 : (double)st.x - log2((double)st.y);
      }
    }
    for (int t0 = 0; t0 < a.w; t0 += TG) {
      __syncthreads();                                       // the previous pass has finished with shared memory
      const int hd = d >> 1;                                 // element pairs per key row
      for (int base = 0; base < TG * hd; base += 4 * NT) {   // four loads in flight per thread before the stores
        raw_t v[4];
        int dst[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int e = base + u * NT + tid;
          const int t = e / hd, cp = e - t * hd;
          const int jj = j - r + t0 + t;
          dst[u] = e < TG * hd ? t * KS + 2 * cp : -1;
          v[u] = raw_t();
          if (e < TG * hd && t0 + t < a.w && jj >= 0 && jj < Le)
            v[u] = *reinterpret_cast<const raw_t*>(kbase + (long long)jj * a.src.k_tok_stride + 2 * cp);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (dst[u] >= 0) *reinterpret_cast<float2*>(ksf + dst[u]) = Pair<T>::to_f32(v[u]);
      }
      double c0 = 0.0, c1 = 0.0, e0 = 0.0, e1 = 0.0;         // two accumulation chains
      for (int cb = 0; cb < d; cb += a.dc) {
        if (cb) __syncthreads();
        const int ncol = min(a.dc, d - cb);
        const int vpr = ncol * (int)sizeof(T) / 16;          // 16-byte vectors per row: copied as they are
        const bool restage = a.dc < d || staged_chunk != c;
        for (int base = 0; restage && base < RB * vpr; base += 4 * NT) {
          uint4 v[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int e = base + u * NT + tid, rr = e / vpr, vc = e - rr * vpr;
            v[u] = make_uint4(0u, 0u, 0u, 0u);
            if (e < RB * vpr && row0 + rr < a.R)
              v[u] = *reinterpret_cast<const uint4*>(qbase + (long long)(row0 + rr) * d + cb + vc * (16 / (int)sizeof(T)));
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int e = base + u * NT + tid, rr = e / vpr, vc = e - rr * vpr;
            if (e < RB * vpr) *reinterpret_cast<uint4*>(qt + rr * q_pitch + vc * 16) = v[u];
          }
        }
        staged_chunk = c;
        __syncthreads();
        const T* qa = reinterpret_cast<const T*>(qt + (wid * 8 + frow) * q_pitch) + fk;   // A fragment: row = lane / 4, column = lane % 4
        const float* kb = ksf + frow * KS + cb + fk;                                   // B fragment: tap = lane / 4, column = lane % 4
#pragma unroll 2
        for (int k0 = 0; k0 < ncol; k0 += 8) {               // ncol is a multiple of 16
          dmma(c0, c1, elem_f64(qa + k0), (double)kb[k0]);
          dmma(e0, e1, elem_f64(qa + k0 + 4), (double)kb[k0 + 4]);
        }
      }
      c0 += e0; c1 += e1;
      // this lane holds the dot products of its row with taps 2 fk and 2 fk + 1
      double wgt[2] = {c0, c1};
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int t = 2 * fk + u, jj = j - r + t0 + t;
        wgt[u] = (row < a.R && t0 + t < a.w && jj >= 0 && jj < Le) ? exp2(fma(wgt[u], a.scale_log2, -mu)) : 0.0;
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) wgt[u] += __shfl_xor_sync(0xffffffffu, wgt[u], o);   // the warp's 8 rows
        if (lane < 4) red[wid][t] = wgt[u];
      }
      __syncthreads();
      if (tid < TG && t0 + tid < a.w) {
        double sum = 0.0;
#pragma unroll
        for (int w2 = 0; w2 < NT / 32; ++w2) sum += red[w2][tid];
        part[((long long)m * chunks + c) * a.w + t0 + tid] = sum;
      }
    }
  }

  // ---- the last CTA of this head to get here ranks the band ----
  __syncthreads();
  if (tid == 0) {
    __threadfence();                                         // this CTA's column sums (ordered before by the barrier) first
    last_s = atomicAdd(&head->done, 1) == (int)gridDim.x - 1;
    __threadfence();
  }
  __syncthreads();
  if (!last_s) return;
  if (overflow) {
    if (tid == 0 && a.status) atomicOr(a.status, SNAP_DEV_BAND_OVERFLOW);
    return;
  }
  const int n_sel = a.K - head->n_sure;                      // band members that belong to the selection
  if (nb == 0 || n_sel < 0 || n_sel > nb) return;            // nothing recorded (or inconsistent): keep the order
  const bool avg = a.pool_mode == SNAP_POOL_AVG;
  float dev = 0.f;
  for (int m = tid; m < nb; m += NT) {
    const int j = band[m].idx_flag & 0x7fffffff;
    double p = avg ? 0.0 : -INFINITY;
    for (int t = 0; t < a.w; ++t) {
      const int jj = j - r + t;
      if (jj < 0 || jj >= Le) continue;
      double cj = 0.0;
      for (int c = 0; c < chunks; ++c) cj += __ldcg(&part[((long long)m * chunks + c) * a.w + t]);
      p = avg ? p + cj : fmax(p, cj);
    }
    if (avg) p /= (double)a.w;
    p64[m] = p;
    jidx[m] = j;
    if (p > 0.0) dev = fmaxf(dev, fabsf((float)((double)band[m].p32 / p - 1.0)));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) dev = fmaxf(dev, __shfl_xor_sync(0xffffffffu, dev, o));
  if (lane == 0) dev_s[wid] = dev;
  if (tid < 2) n_list[tid] = 0;
  __syncthreads();
  for (int m = tid; m < nb; m += NT) {
    const int e = band[m].idx_flag, j = e & 0x7fffffff;
    const double p = p64[m];
    int rank = 0;
    for (int o = 0; o < nb; ++o) {
      const double po = p64[o];
      rank += po > p || (po == p && jidx[o] < j);
    }
    const bool sel64 = rank < n_sel, sel32 = e < 0;
    if (sel32 != sel64) lists[sel64][atomicAdd(&n_list[sel64], 1)] = j;
  }
  __syncthreads();
  for (int m = tid; m < nb; m += NT) part[(long long)m * chunks * a.w] = p64[m];   // left in scratch for diagnosis
  const int n_out = n_list[0], n_in = n_list[1];
  // the verdict for the gather kernel: how many positions change places, and which
  const bool ok = n_in == n_out;
  int* glists = rf.lists + (long long)z * 2 * rf.cap;
  for (int u = tid; u < (ok ? n_in : 0); u += NT) {
    glists[u] = lists[0][u];
    glists[rf.cap + u] = lists[1][u];
  }
  if (tid == 0) {
    float dmax = 0.f;
    for (int w2 = 0; w2 < NT / 32; ++w2) dmax = fmaxf(dmax, dev_s[w2]);
    head->max_dev = dmax;
    head->changed = ok ? n_in : 0;
  }
}

}  // namespace

int refine_row_chunks(const Shape& s) { return (s.g * s.Lo + RB - 1) / RB; }

cudaError_t launch_topk_refine(int dtype, const Shape& s, const SeqBatch& b, const void* q_obs, const KVSource& src,
                               const ScoreBuffers& buf, uint32_t* status, int sm_count, cudaStream_t st) {
  if (!buf.ref.head || b.n_scored == 0 || s.K == 0) return cudaSuccess;
  RefineArgs a;
  a.q = q_obs; a.src = src;
  a.Hq = s.Hq; a.Hkv = s.Hkv; a.g = s.g; a.Lo = s.Lo; a.d = s.d_qk; a.Ls = s.Ls; a.Lr = s.Lr; a.K = s.K;
  a.w = s.w; a.pool_mode = s.pool_mode; a.R = s.g * s.Lo;
  a.elt = dtype == SNAP_F32 ? 4 : 2;
  a.scale_log2 = (double)s.scale * 1.4426950408889634074;
  a.b = b; a.buf = buf; a.status = status;
  const int nz = b.n_scored * s.Hkv;
  int gx = (2 * sm_count + nz - 1) / nz;                     // CTAs per head (two per SM in all); each takes a run of the head's items
  gx = gx < 1 ? 1 : gx > 1024 ? 1024 : gx;
  // columns staged at a time: the whole row when 64 rows of it fit the tile, else the largest multiple of 16 that does
  const int max_cols = (QTILE_B / RB - 16) / a.elt / 16 * 16;
  a.dc = s.d_qk < max_cols ? s.d_qk : max_cols;
  const size_t smem = (size_t)TG * (s.d_qk + 4) * sizeof(float) + (size_t)RB * (a.dc * a.elt + 16);
  static SmemLimit lim_f = {}, lim_b = {};
  cudaError_t e;
  if (dtype == SNAP_F32) {
    if ((e = ensure_dyn_smem(topk_refine_kernel<float>, smem, lim_f)) != cudaSuccess) return e;
    e = launch_pdl(topk_refine_kernel<float>, dim3(gx, nz), dim3(NT), smem, st, a);
  } else {
    if ((e = ensure_dyn_smem(topk_refine_kernel<__nv_bfloat16>, smem, lim_b)) != cudaSuccess) return e;
    e = launch_pdl(topk_refine_kernel<__nv_bfloat16>, dim3(gx, nz), dim3(NT), smem, st, a);
  }
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace snap
