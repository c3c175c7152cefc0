// Sequence-axis pooling and per-KV-head top-K (Eq. 2), one CTA per (prompt, KV head).
//
//   P[j] = pool_w(C)[j]  (1-D, stride 1, pad w/2; average divides by w over zero padding, max pads -inf)
//   keep the K largest P, ties to the lower index, and emit absolute positions in ascending order.
//
// Selection is an 8-bit-digit radix select on the order-preserving integer image of P (four
// histogram passes narrow down the K-th largest key), followed by an ordered compaction: every
// key above the threshold is taken, and of the keys equal to it the first ones in index order
// until K are reached.  Histograms are per-warp in shared memory, bin search is one warp's
// shuffle scan, and the compaction uses warp ballots, so no global atomics are involved.
// Prompts with at most K candidates keep them all and skip scoring altogether.
#include "snap_internal.cuh"

namespace snap {
namespace {

constexpr int NT = 1024, NW = NT / 32;

struct TopkArgs {
  int Hkv, Ls, Lr, K, w, pool_mode;
  SeqBatch b;
  ScoreBuffers buf;
  int* idx_out;      // [n][Hkv][K]
};

__device__ __forceinline__ unsigned key_of(float x) {
  const unsigned u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Exclusive prefix of a 0/1 flag over the whole CTA (thread order), plus the CTA total.
// warp_tot is a shared array of NW+1 ints.  Two barriers.
__device__ __forceinline__ int block_rank(bool flag, int* warp_tot, int& total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const unsigned bal = __ballot_sync(0xffffffffu, flag);
  if (lane == 0) warp_tot[wid] = __popc(bal);
  __syncthreads();
  if (wid == 0) {
    const int v = warp_tot[lane];
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += n;
    }
    warp_tot[lane] = inc - v;
    if (lane == 31) warp_tot[NW] = inc;
  }
  __syncthreads();
  const int r = warp_tot[wid] + __popc(bal & ((1u << lane) - 1u));
  total = warp_tot[NW];
  __syncthreads();
  return r;
}

__global__ void __launch_bounds__(NT) pool_topk_kernel(const TopkArgs a) {
  __shared__ int hist[NW][256];
  __shared__ int bins[256];
  __shared__ int warp_tot[NW + 1];
  __shared__ unsigned sh_prefix;
  __shared__ int sh_remaining;

  const int seq = blockIdx.y, kvh = blockIdx.x;
  const int L = a.b.len[seq];
  const int Le = L - a.Ls - a.Lr;
  const int K = a.K;
  int* out = a.idx_out + ((long long)(a.b.first_seq + seq) * a.Hkv + kvh) * K;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;

  if (Le <= K || a.b.score_idx[seq] < 0) {           // keep every candidate (or none)
    const int nv = max(min(Le, K), 0);
    for (int i = tid; i < K; i += NT) out[i] = i < nv ? a.Ls + i : -1;
    return;
  }

  const long long zoff = ((long long)a.b.score_idx[seq] * a.Hkv + kvh) * a.buf.c_stride;
  const float* __restrict__ C = a.buf.C + zoff;
  float* __restrict__ P = a.buf.P + zoff;

  // ---- pooling ----
  const int r = a.w / 2;
  if (a.pool_mode == SNAP_POOL_AVG) {
    const float inv_w = 1.0f / (float)a.w;
    for (int j = tid; j < Le; j += NT) {
      float s = 0.f;
      for (int t = -r; t <= r; ++t) {
        const int jj = j + t;
        if (jj >= 0 && jj < Le) s += C[jj];
      }
      P[j] = s * inv_w;
    }
  } else {
    for (int j = tid; j < Le; j += NT) {
      float s = -INFINITY;
      for (int t = -r; t <= r; ++t) {
        const int jj = j + t;
        if (jj >= 0 && jj < Le) s = fmaxf(s, C[jj]);
      }
      P[j] = s;
    }
  }
  if (tid == 0) { sh_prefix = 0u; sh_remaining = K; }
  __syncthreads();

  // ---- radix select of the K-th largest key ----
  unsigned mask = 0u;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = tid; i < NW * 256; i += NT) (&hist[0][0])[i] = 0;
    __syncthreads();
    const unsigned prefix = sh_prefix;
    for (int j = tid; j < Le; j += NT) {
      const unsigned key = key_of(P[j]);
      if ((key & mask) == prefix) atomicAdd(&hist[wid][(key >> shift) & 255u], 1);
    }
    __syncthreads();
    if (tid < 256) {
      int s = 0;
#pragma unroll 8
      for (int w2 = 0; w2 < NW; ++w2) s += hist[w2][tid];
      bins[tid] = s;
    }
    __syncthreads();
    if (wid == 0) {
      // lane l owns bins 255-8l .. 248-8l (descending); find the bin holding the remaining-th largest
      const int remaining = sh_remaining;
      int loc[8], csum = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) { loc[i] = bins[255 - 8 * lane - i]; csum += loc[i]; }
      int inc = csum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
      }
      int excl = inc - csum;
      if (excl < remaining && remaining <= inc) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (excl + loc[i] >= remaining) {
            sh_prefix = prefix | ((unsigned)(255 - 8 * lane - i) << shift);
            sh_remaining = remaining - excl;
            break;
          }
          excl += loc[i];
        }
      }
    }
    mask |= 255u << shift;
    __syncthreads();
  }
  const unsigned tau = sh_prefix;      // key of the K-th largest pooled score
  const int need_eq = sh_remaining;    // how many keys equal to tau are taken (>= 1)
  __syncthreads();

  // ---- ordered emission ----
  int run_eq = 0, run_out = 0;
  for (int base = 0; base < Le; base += NT) {
    const int j = base + tid;
    unsigned key = 0u;
    if (j < Le) key = key_of(P[j]);
    const bool gt = j < Le && key > tau;
    const bool eq = j < Le && key == tau;
    int tot_eq, tot_sel;
    const int rank_eq = block_rank(eq, warp_tot, tot_eq);
    const bool sel = gt || (eq && run_eq + rank_eq < need_eq);
    const int rank_sel = block_rank(sel, warp_tot, tot_sel);
    if (sel) out[run_out + rank_sel] = a.Ls + j;
    run_eq += tot_eq;
    run_out += tot_sel;
  }
}

}  // namespace

cudaError_t launch_pool_topk(const Shape& s, const SeqBatch& b, const ScoreBuffers& buf,
                             int* idx_out, uint32_t* status, cudaStream_t st) {
  (void)status;
  if (s.K == 0 || b.n == 0) return cudaSuccess;
  TopkArgs a;
  a.Hkv = s.Hkv; a.Ls = s.Ls; a.Lr = s.Lr; a.K = s.K; a.w = s.w; a.pool_mode = s.pool_mode;
  a.b = b; a.buf = buf; a.idx_out = idx_out;
  dim3 grid(s.Hkv, b.n);
  pool_topk_kernel<<<grid, NT, 0, st>>>(a);
  count_launch();
  return cudaGetLastError();
}

}  // namespace snap
