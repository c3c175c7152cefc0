// Causal prefill attention that also emits the normalisers of Eq. 4, portable version: any
// element type, head sizes and group size, the latent layout included (V = the first d_v
// elements of the K row).  It serves the layers the tensor-core kernel does not take (fp32, head
// sizes other than 128, the latent layout); it is written for coverage, not for speed.
//
// One warp per (query position t, head): it walks the keys 0..t in tiles of 32, lane r owning
// key r of the tile.  A logit is a dot product spread over the lanes (lane c holds elements
// c, c + 32, ... of the query row in registers) and reduced with shuffles; the tile's 32 logits
// update the running max / sum (online softmax, natural exponentials in fp32), and every lane
// accumulates p.V for the output elements it owns.  Rows of the last Lo positions also sum the
// same exponentials over the eviction candidates [Ls, L - Lr) alone: max + log of that sum, in
// base 2, is what Eq. 4 divides by.  The four warps of a CTA take consecutive positions of one
// head, so that they read the same key and value rows at about the same time.
#include "snap_internal.cuh"

namespace snap {
namespace {

constexpr int NT = 128, NW = NT / 32, TK = 32, MAXQ = 32, MAXC = 16;   // d_qk <= 1024, d_v <= 512

struct GArgs {
  const void* q; const void* k; const void* v;
  long long k_tok, k_head, v_tok, v_head;     // elements
  SeqBatch b;
  int Hq, g, d_qk, d_v, Ls, Lr, Lo;
  float scale;
  void* out;
  float* mu;
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

template <typename T>
__global__ void __launch_bounds__(NT) prefill_generic_kernel(const GArgs a) {
  const int seq = blockIdx.z, head = blockIdx.y, lane = threadIdx.x & 31;
  const int L = a.b.len[seq];
  const int t = blockIdx.x * NW + (threadIdx.x >> 5);          // this warp's query position
  if (t >= L) return;
  const int tok0 = a.b.tok_off[seq], kvh = head / a.g;
  const T* qrow = static_cast<const T*>(a.q) + ((long long)(tok0 + t) * a.Hq + head) * a.d_qk;
  const T* kbase = static_cast<const T*>(a.k) + (long long)tok0 * a.k_tok + (long long)kvh * a.k_head;
  const T* vbase = static_cast<const T*>(a.v) + (long long)tok0 * a.v_tok + (long long)kvh * a.v_head;

  float qreg[MAXQ], acc[MAXC];
#pragma unroll
  for (int i = 0; i < MAXQ; ++i) qreg[i] = lane + 32 * i < a.d_qk ? to_f32<T>(qrow[lane + 32 * i]) : 0.f;
#pragma unroll
  for (int i = 0; i < MAXC; ++i) acc[i] = 0.f;
  const bool window = a.mu != nullptr && t >= L - a.Lo;
  const int cand_lo = a.Ls, cand_hi = L - a.Lr;                // candidates [cand_lo, cand_hi)
  float m = -INFINITY, l = 0.f, lc = 0.f;

  for (int j0 = 0; j0 <= t; j0 += TK) {
    const int nk = min(TK, t + 1 - j0);                        // keys of this tile the row may see
    float s_mine = -INFINITY;
    for (int r = 0; r < nk; ++r) {
      const T* krow = kbase + (long long)(j0 + r) * a.k_tok;
      float part = 0.f;
#pragma unroll
      for (int i = 0; i < MAXQ; ++i)
        if (32 * i < a.d_qk && lane + 32 * i < a.d_qk) part = fmaf(qreg[i], to_f32<T>(krow[lane + 32 * i]), part);
      const float s = warp_sum(part) * a.scale;
      if (lane == r) s_mine = s;
    }
    const float m_new = fmaxf(m, warp_max(s_mine));
    const float alpha = m == -INFINITY ? 0.f : expf(m - m_new);
    const float p = lane < nk ? expf(s_mine - m_new) : 0.f;
    l = l * alpha + warp_sum(p);
    if (window) {
      const int j = j0 + lane;
      lc = lc * alpha + warp_sum(j >= cand_lo && j < cand_hi ? p : 0.f);
    }
    m = m_new;
#pragma unroll
    for (int i = 0; i < MAXC; ++i) acc[i] *= alpha;
    for (int r = 0; r < nk; ++r) {
      const float pr = __shfl_sync(0xffffffffu, p, r);
      const T* vrow = vbase + (long long)(j0 + r) * a.v_tok;
#pragma unroll
      for (int i = 0; i < MAXC; ++i)
        if (32 * i < a.d_v && lane + 32 * i < a.d_v) acc[i] = fmaf(pr, to_f32<T>(vrow[lane + 32 * i]), acc[i]);
    }
  }
  const float inv = 1.f / l;
  T* orow = static_cast<T*>(a.out) + ((long long)(tok0 + t) * a.Hq + head) * a.d_v;
#pragma unroll
  for (int i = 0; i < MAXC; ++i)
    if (lane + 32 * i < a.d_v) orow[lane + 32 * i] = from_f32<T>(acc[i] * inv);
  if (window && lane == 0)
    a.mu[((long long)(a.b.first_seq + seq) * a.Hq + head) * a.Lo + (t - (L - a.Lo))] =
        lc > 0.f ? (m + logf(lc)) * 1.4426950408889634f : -INFINITY;
}

}  // namespace

cudaError_t launch_prefill_generic(int dtype, const Shape& s, const SeqBatch& b, const void* q, const KVSource& src,
                                   void* out, float* mu, cudaStream_t st) {
  int max_len = 0;
  for (int i = 0; i < b.n; ++i) max_len = max_len > b.len[i] ? max_len : b.len[i];
  if (b.n == 0 || max_len == 0) return cudaSuccess;
  GArgs a;
  a.q = q; a.k = src.k;
  a.k_tok = src.k_tok_stride; a.k_head = src.k_head_stride;
  if (s.v_aliases_k) { a.v = src.k; a.v_tok = src.k_tok_stride; a.v_head = src.k_head_stride; }
  else { a.v = src.v; a.v_tok = src.v_tok_stride; a.v_head = src.v_head_stride; }
  a.b = b;
  a.Hq = s.Hq; a.g = s.g; a.d_qk = s.d_qk; a.d_v = s.d_v; a.Ls = s.Ls; a.Lr = s.Lr; a.Lo = s.Lo;
  a.scale = s.scale;
  a.out = out; a.mu = mu;
  const dim3 grid((max_len + NW - 1) / NW, s.Hq, b.n);
  if (dtype == SNAP_F32) prefill_generic_kernel<float><<<grid, NT, 0, st>>>(a);
  else prefill_generic_kernel<__nv_bfloat16><<<grid, NT, 0, st>>>(a);
  count_launch();
  return cudaGetLastError();
}

}  // namespace snap
