// Observation-window scores, portable SIMT version (any element type, any head size).
//
// Computes, for every scored prompt and KV head, Eq. 1's column sums of Eq. 4's softmax:
//   C[j] = sum over the g query heads of the KV head, over the Lo window rows i, of
//          exp(scale * q_i . k_j - m_i) / l_i ,      j over the eviction candidates [Ls, L - Lr)
// in two passes, because every row's normaliser l_i must be known before any column sum:
//   pass 1  row statistics (running max m_i, sum of exponentials l_i) per candidate split,
//           merged across splits in double precision;
//   pass 2  recomputes the logits and accumulates the normalised column sums.
// This version is used for fp32 inputs and as the fallback for shapes the tensor-core
// version does not cover.  Tiles: 64 query rows x 64 candidates, 16-deep k slices, 4x4 per thread.
#include "snap_internal.cuh"

namespace snap {
namespace {

constexpr int BM = 64, BN = 64, BK = 16, NT = 256;

struct ScoreArgs {
  const void* q;
  const void* k;
  long long k_tok_stride, k_head_stride;
  int Hq, Hkv, g, Lo, d, Ls, Lr;
  float scale;
  SeqBatch b;
  ScoreBuffers buf;
};

template <typename T>
__device__ __forceinline__ void tile_scores(const T* __restrict__ qbase, const T* __restrict__ kbase,
                                            long long tok_stride, int d, int R, int Le, int row0,
                                            int cand0, float (&acc)[4][4], float (*As)[BM + 4],
                                            float (*Bs)[BN + 4]) {
  const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  const int lr = tid / 4, lk = (tid % 4) * 4;
  const bool a_ok = row0 + lr < R, b_ok = cand0 + lr < Le;
  const T* ap = qbase + (long long)(row0 + lr) * d + lk;
  const T* bp = kbase + (long long)(cand0 + lr) * tok_stride + lk;
  for (int k0 = 0; k0 < d; k0 += BK) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      As[lk + i][lr] = a_ok ? to_f32<T>(ap[k0 + i]) : 0.f;
      Bs[lk + i][lr] = b_ok ? to_f32<T>(bp[k0 + i]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      const float4 a4 = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
      const float4 b4 = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
      const float av[4] = {a4.x, a4.y, a4.z, a4.w}, bv[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
}

__device__ __forceinline__ float half_warp_max(float v) {
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float half_warp_sum(float v) {
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Pass 1: per (candidate split, 64-row block, scored prompt x KV head).
template <typename T>
__global__ void __launch_bounds__(NT) score_stats_kernel(const ScoreArgs a) {
  __shared__ __align__(16) float As[BK][BM + 4];
  __shared__ __align__(16) float Bs[BK][BN + 4];
  const int z = blockIdx.z, si = z / a.Hkv, kvh = z % a.Hkv;
  const int seq = a.b.seq_of_score[si];
  const int Le = a.b.len[seq] - a.Ls - a.Lr;
  const int R = a.g * a.Lo;
  const int row0 = blockIdx.y * BM;
  if (row0 >= R) return;
  const int ntiles = (Le + BN - 1) / BN;
  const int tps = (ntiles + a.buf.nsplit - 1) / a.buf.nsplit;
  const int t0 = blockIdx.x * tps, t1 = min(ntiles, t0 + tps);
  const T* qbase = static_cast<const T*>(a.q) +
                   ((long long)(a.b.first_seq + seq) * a.Hq + (long long)kvh * a.g) * a.Lo * a.d;
  const T* kbase = static_cast<const T*>(a.k) + (long long)(a.b.tok_off[seq] + a.Ls) * a.k_tok_stride +
                   (long long)kvh * a.k_head_stride;
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  float m_run[4], l_run[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) { m_run[i] = -INFINITY; l_run[i] = 0.f; }
  float acc[4][4];
  for (int t = t0; t < t1; ++t) {
    const int cand0 = t * BN;
    tile_scores<T>(qbase, kbase, a.k_tok_stride, a.d, R, Le, row0, cand0, acc, As, Bs);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float tmax = -INFINITY;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        acc[i][j] *= a.scale;
        if (cand0 + tx * 4 + j < Le) tmax = fmaxf(tmax, acc[i][j]);
      }
      tmax = half_warp_max(tmax);
      const float m_new = fmaxf(m_run[i], tmax);
      float sum = 0.f;
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (cand0 + tx * 4 + j < Le) sum += expf(acc[i][j] - m_new);
      sum = half_warp_sum(sum);
      l_run[i] = l_run[i] * expf(m_run[i] - m_new) + sum;
      m_run[i] = m_new;
    }
  }
  if (tx == 0) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int row = row0 + ty * 4 + i;
      if (row < R)
        a.buf.part_stats[((long long)z * a.buf.nsplit + blockIdx.x) * R + row] =
            make_float2(m_run[i], l_run[i]);
    }
  }
}

// Merge the per-split statistics: m = max_s m_s, l = sum_s l_s exp(m_s - m), kept as (m, 1/l).
// One warp per query row, lanes over the splits (a thread per row walking the splits one dependent load and
// one double-precision exponential at a time took 18 us for 60 splits).
__global__ void score_combine_kernel(const float2* __restrict__ part, float2* __restrict__ stats,
                                     double* __restrict__ mu64, int nsplit, int R) {
  const long long z = blockIdx.y;
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= R) return;
  float m = -INFINITY;
  for (int s = lane; s < nsplit; s += 32) m = fmaxf(m, part[(z * nsplit + s) * R + row].x);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  double l = 0.0;
  for (int s = lane; s < nsplit; s += 32) {
    const float2 p = part[(z * nsplit + s) * R + row];
    if (p.y > 0.f) l += (double)p.y * exp((double)p.x - (double)m);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
  if (lane == 0) {
    stats[z * R + row] = make_float2(m, (float)(1.0 / l));
    if (mu64) mu64[z * R + row] = ((double)m + log(l)) * 1.4426950408889634074;   // log2 domain, unrounded
  }
}

// Pass 2: per (candidate tile, scored prompt x KV head); loops over all query-row blocks.
template <typename T>
__global__ void __launch_bounds__(NT) score_colsum_kernel(const ScoreArgs a) {
  __shared__ __align__(16) float As[BK][BM + 4];
  __shared__ __align__(16) float Bs[BK][BN + 4];
  __shared__ float2 st[BM];
  __shared__ float red[16][BN];
  const int z = blockIdx.z, si = z / a.Hkv, kvh = z % a.Hkv;
  const int seq = a.b.seq_of_score[si];
  const int Le = a.b.len[seq] - a.Ls - a.Lr;
  const int R = a.g * a.Lo;
  const int cand0 = blockIdx.x * BN;
  if (cand0 >= Le) return;
  const T* qbase = static_cast<const T*>(a.q) +
                   ((long long)(a.b.first_seq + seq) * a.Hq + (long long)kvh * a.g) * a.Lo * a.d;
  const T* kbase = static_cast<const T*>(a.k) + (long long)(a.b.tok_off[seq] + a.Ls) * a.k_tok_stride +
                   (long long)kvh * a.k_head_stride;
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  float col[4] = {0.f, 0.f, 0.f, 0.f};
  float acc[4][4];
  for (int row0 = 0; row0 < R; row0 += BM) {
    if (threadIdx.x < BM) {
      const int row = row0 + threadIdx.x;
      if (row >= R) st[threadIdx.x] = make_float2(0.f, 0.f);
      else if (a.buf.ext_mu)                                   // log2 normaliser from outside: (m, 1/l) = (mu ln 2, 1)
        st[threadIdx.x] = make_float2(
            a.buf.ext_mu[((long long)(a.b.first_seq + seq) * a.Hq + (long long)kvh * a.g) * a.Lo + row] * 0.6931471805599453f, 1.f);
      else st[threadIdx.x] = a.buf.stats[(long long)z * R + row];
    }
    tile_scores<T>(qbase, kbase, a.k_tok_stride, a.d, R, Le, row0, cand0, acc, As, Bs);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 s = st[ty * 4 + i];
      if (row0 + ty * 4 + i < R) {
#pragma unroll
        for (int j = 0; j < 4; ++j) col[j] += expf(acc[i][j] * a.scale - s.x) * s.y;
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) red[ty][tx * 4 + j] = col[j];
  __syncthreads();
  if (threadIdx.x < BN && cand0 + threadIdx.x < Le) {
    float s = 0.f;
#pragma unroll
    for (int r = 0; r < 16; ++r) s += red[r][threadIdx.x];
    a.buf.C[(long long)z * a.buf.c_stride + cand0 + threadIdx.x] = s;
  }
}

template <typename T>
cudaError_t launch_t(const ScoreArgs& a, int max_le, cudaStream_t st) {
  const int R = a.g * a.Lo;
  const int nz = a.b.n_scored * a.Hkv;
  if (!a.buf.ext_mu) {                                        // Eq. 4's normalisers, unless the caller has them
    dim3 g1(a.buf.nsplit, (R + BM - 1) / BM, nz);
    score_stats_kernel<T><<<g1, NT, 0, st>>>(a);
    count_launch();
    score_combine_kernel<<<dim3((R + 7) / 8, nz), 256, 0, st>>>(a.buf.part_stats, a.buf.stats, a.buf.ref.mu64, a.buf.nsplit, R);
    count_launch();
  }
  dim3 g2((max_le + BN - 1) / BN, 1, nz);
  score_colsum_kernel<T><<<g2, NT, 0, st>>>(a);
  count_launch();
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_score_simt(int dtype, const Shape& s, const SeqBatch& b, const void* q_obs,
                              const KVSource& src, const ScoreBuffers& buf, cudaStream_t st) {
  if (b.n_scored == 0) return cudaSuccess;
  ScoreArgs a;
  a.q = q_obs; a.k = src.k; a.k_tok_stride = src.k_tok_stride; a.k_head_stride = src.k_head_stride;
  a.Hq = s.Hq; a.Hkv = s.Hkv; a.g = s.g; a.Lo = s.Lo; a.d = s.d_qk; a.Ls = s.Ls; a.Lr = s.Lr;
  a.scale = s.scale; a.b = b; a.buf = buf;
  int max_le = 0;
  for (int i = 0; i < b.n; ++i)
    if (b.score_idx[i] >= 0) max_le = max(max_le, b.len[i] - s.Ls - s.Lr);
  if (dtype == SNAP_F32) return launch_t<float>(a, max_le, st);
  return launch_t<__nv_bfloat16>(a, max_le, st);
}

}  // namespace snap
