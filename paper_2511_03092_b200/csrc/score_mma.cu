// Observation-window scores on the tensor cores (Eq. 4 -> Eq. 1 with the GQA group sum), for
// bf16 layers with 128-wide heads and at most 256 window rows per KV head (g * Lo <= 256).
//
// The only dense contraction of the method: S^T = K_evict . Q_obs^T, with M = candidates and
// N = the g*Lo query rows of one KV head.  A CTA keeps the whole query block in shared memory
// and streams 64-candidate key tiles through a two-stage cp.async ring (16-byte chunks,
// XOR-swizzled so that ldmatrix is conflict free); warp w owns query rows [32w, 32w+32) and
// all 64 candidates of the tile, so every softmax statistic stays inside one warp:
//
//   pass 1  running (reference max, sum of exp2) per query row, kept per thread over the CTA's
//           run of tiles and merged across the 8 lanes that share a row at the end.  The
//           reference is refreshed lazily: only when a tile's partial sum shows a logit far
//           above it.
//   pass 2  recomputes the logits and forms, per candidate, sum_i exp2(s_ij - m_i) / l_i over
//           the thread's 8 rows, then over the quad, then over the warps through shared memory.
//
// mma.sync.m16n8k16 (bf16 in, fp32 accumulate) is the instruction used here; statistics are in
// the log2 domain (logits are multiplied by scale * log2 e once).
#include "mma_helpers.cuh"
#include "snap_internal.cuh"

namespace snap {
namespace {

using namespace mmasync;

constexpr int D = 128, TN = 64, ROW_B = D * 2, KT_B = TN * ROW_B;

struct MmaArgs {
  const __nv_bfloat16* q; const __nv_bfloat16* k;
  long long k_tok_b, k_head_b;       // bytes
  int Hq, Hkv, g, Lo, Ls, Lr, R, RP; // R = g*Lo query rows, RP = R padded to a multiple of 32
  float scale_log2;
  SeqBatch b;
  ScoreBuffers buf;
};

// rows x 256 bytes, 16-byte chunk c of row r stored at chunk c ^ (r & 7)
__device__ __forceinline__ uint32_t swz(int row, int chunk) { return row * ROW_B + ((chunk ^ (row & 7)) << 4); }

__device__ __forceinline__ void load_k_tile(uint32_t dst, const char* kbase, long long tok_b, int cand0, int Le) {
  for (int idx = threadIdx.x; idx < TN * 16; idx += blockDim.x) {
    const int r = idx >> 4, c = idx & 15;
    const bool ok = cand0 + r < Le;
    const char* src = ok ? kbase + (long long)(cand0 + r) * tok_b + c * 16 : kbase;
    cp_async16(dst + swz(r, c), src, ok ? 16u : 0u);
  }
}

// merge two (reference max, sum) pairs of the log2 domain
__device__ __forceinline__ void merge_ml(float& m, float& l, float m2, float l2) {
  const float mn = fmaxf(m, m2);
  const float f1 = m == -INFINITY ? 0.f : exp2f(m - mn), f2 = m2 == -INFINITY ? 0.f : exp2f(m2 - mn);
  l = l * f1 + l2 * f2;
  m = mn;
}

template <int PASS>
__global__ void __launch_bounds__(256, 2) score_mma_kernel(const MmaArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int NRW = blockDim.x >> 5;
  unsigned char* Qs = smem;                                 // [RP][256 B]
  unsigned char* Ks = Qs + a.RP * ROW_B;                    // [2][64][256 B]
  float* colpart = reinterpret_cast<float*>(Ks + 2 * KT_B); // [2][NRW][64]  (pass 2)

  const int z = blockIdx.y, si = z / a.Hkv, kvh = z % a.Hkv;
  const int seq = a.b.seq_of_score[si];
  const int Le = a.b.len[seq] - a.Ls - a.Lr;
  const int R = a.R;
  const int ntiles = (Le + TN - 1) / TN;
  const int t0 = (int)((long long)ntiles * blockIdx.x / a.buf.nsplit);
  const int t1 = (int)((long long)ntiles * (blockIdx.x + 1) / a.buf.nsplit);
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  const __nv_bfloat16* qbase = a.q + ((long long)(a.b.first_seq + seq) * a.Hq + (long long)kvh * a.g) * a.Lo * D;
  const char* kbase = reinterpret_cast<const char*>(a.k) + (long long)(a.b.tok_off[seq] + a.Ls) * a.k_tok_b +
                      (long long)kvh * a.k_head_b;
  const uint32_t qs = smem_u32(Qs), ks0 = smem_u32(Ks);

  // the thread's 8 query rows: n-tile t (0..3), element e (0..1) -> row 32w + 8t + 2(lane%4) + e
  float cm[8], cl[8];      // pass 1: running reference max / sum;  pass 2: m_i / (1/l_i)
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    const int row = 32 * w + 8 * (c >> 1) + 2 * (lane & 3) + (c & 1);
    if (PASS == 1) { cm[c] = -INFINITY; cl[c] = 0.f; }
    else {
      float2 st = make_float2(0.f, 0.f);
      if (row < R)
        st = a.buf.ext_mu   // log2 normaliser from outside: (m, 1/l) = (mu, 1)
                 ? make_float2(a.buf.ext_mu[((long long)(a.b.first_seq + seq) * a.Hq + (long long)kvh * a.g) * a.Lo + row], 1.f)
                 : a.buf.stats[(long long)z * R + row];
      cm[c] = st.x; cl[c] = st.y;
    }
  }
  if (t0 >= t1) {                                           // nothing to do for this split
    if (PASS == 1 && (lane >> 2) == 0) {
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const int row = 32 * w + 8 * (c >> 1) + 2 * (lane & 3) + (c & 1);
        if (row < R) a.buf.part_stats[((long long)z * a.buf.nsplit + blockIdx.x) * R + row] = make_float2(-INFINITY, 0.f);
      }
    }
    return;
  }

  for (int idx = tid; idx < a.RP * 16; idx += blockDim.x) {
    const int r = idx >> 4, c = idx & 15;
    const bool ok = r < R;
    cp_async16(qs + swz(r, c), ok ? reinterpret_cast<const char*>(qbase) + (long long)r * ROW_B + c * 16
                                  : reinterpret_cast<const char*>(qbase), ok ? 16u : 0u);
  }
  load_k_tile(ks0, kbase, a.k_tok_b, t0 * TN, Le);
  cp_commit();

  // per-lane ldmatrix coordinates
  const int a_row = (lane & 7) + ((lane >> 3) & 1) * 8, a_chk = lane >> 4;       // + 16*mt, + 2*ks
  const int b_row = 32 * w + (lane & 7) + (lane >> 4) * 8, b_chk = (lane >> 3) & 1;  // + 16*np, + 2*ks

  for (int t = t0; t < t1; ++t) {
    const int stage = (t - t0) & 1;
    if (t + 1 < t1) {
      load_k_tile(ks0 + (stage ^ 1) * KT_B, kbase, a.k_tok_b, (t + 1) * TN, Le);
      cp_commit();
      cp_wait<1>();
    } else {
      cp_wait<0>();
    }
    __syncthreads();

    float acc[4][4][4];                                     // [m-tile][n-tile][frag]
#pragma unroll
    for (int mt = 0; mt < 4; ++mt)
#pragma unroll
      for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int f = 0; f < 4; ++f) acc[mt][nt][f] = 0.f;
    const uint32_t kst = ks0 + stage * KT_B;
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
      uint32_t bq[2][4];
#pragma unroll
      for (int np = 0; np < 2; ++np)
        ldsm4(qs + swz(b_row + 16 * np, 2 * ks + b_chk), bq[np][0], bq[np][1], bq[np][2], bq[np][3]);
#pragma unroll
      for (int mt = 0; mt < 4; ++mt) {
        uint32_t af[4];
        ldsm4(kst + swz(a_row + 16 * mt, 2 * ks + a_chk), af[0], af[1], af[2], af[3]);
#pragma unroll
        for (int np = 0; np < 2; ++np) {
          mma16816(acc[mt][2 * np], af, bq[np][0], bq[np][1]);
          mma16816(acc[mt][2 * np + 1], af, bq[np][2], bq[np][3]);
        }
      }
    }

    // candidates held by this thread: m-tile mt, half hf -> cand0 + 16mt + lane/4 + 8hf
    const int cand0 = t * TN;
    const bool full = cand0 + TN <= Le;
    const int crow = cand0 + (lane >> 2);
    if (PASS == 1) {
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const int nt = c >> 1, e = c & 1;
        float sum = 0.f;
#pragma unroll
        for (int mt = 0; mt < 4; ++mt)
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
            const float ex = exp2f(fmaf(acc[mt][nt][2 * hf + e], a.scale_log2, -cm[c]));
            sum += (full || crow + 16 * mt + 8 * hf < Le) ? ex : 0.f;
          }
        if (!(sum < 4096.f)) {                              // a logit far above the reference (or first tile)
          float vmax = -INFINITY;
#pragma unroll
          for (int mt = 0; mt < 4; ++mt)
#pragma unroll
            for (int hf = 0; hf < 2; ++hf)
              if (full || crow + 16 * mt + 8 * hf < Le) vmax = fmaxf(vmax, acc[mt][nt][2 * hf + e] * a.scale_log2);
          const float mn = fmaxf(cm[c], vmax);
          if (mn != -INFINITY) {
            cl[c] *= cm[c] == -INFINITY ? 0.f : exp2f(cm[c] - mn);
            cm[c] = mn;
            sum = 0.f;
#pragma unroll
            for (int mt = 0; mt < 4; ++mt)
#pragma unroll
              for (int hf = 0; hf < 2; ++hf)
                if (full || crow + 16 * mt + 8 * hf < Le)
                  sum += exp2f(fmaf(acc[mt][nt][2 * hf + e], a.scale_log2, -mn));
          } else {
            sum = 0.f;
          }
        }
        cl[c] += sum;
      }
    } else {
      float csum[8];                                        // [mt*2 + hf]
#pragma unroll
      for (int mt = 0; mt < 4; ++mt)
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          float s = 0.f;
#pragma unroll
          for (int c = 0; c < 8; ++c)
            s = fmaf(exp2f(fmaf(acc[mt][c >> 1][2 * hf + (c & 1)], a.scale_log2, -cm[c])), cl[c], s);
          s += __shfl_xor_sync(0xffffffffu, s, 1);
          s += __shfl_xor_sync(0xffffffffu, s, 2);
          csum[mt * 2 + hf] = s;
        }
      float* cp = colpart + ((stage * NRW + w) * TN);
      if ((lane & 3) == 0) {
#pragma unroll
        for (int mt = 0; mt < 4; ++mt)
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) cp[16 * mt + 8 * hf + (lane >> 2)] = csum[mt * 2 + hf];
      }
    }
    __syncthreads();
    if (PASS == 2) {
      for (int cc = tid; cc < TN && cand0 + cc < Le; cc += blockDim.x) {
        float s = 0.f;
        for (int ww = 0; ww < NRW; ++ww) s += colpart[(stage * NRW + ww) * TN + cc];
        a.buf.C[(long long)z * a.buf.c_stride + cand0 + cc] = s;
      }
    }
  }

  if (PASS == 1) {
#pragma unroll
    for (int c = 0; c < 8; ++c) {
#pragma unroll
      for (int o = 4; o <= 16; o <<= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, cm[c], o);
        const float l2 = __shfl_xor_sync(0xffffffffu, cl[c], o);
        merge_ml(cm[c], cl[c], m2, l2);
      }
      const int row = 32 * w + 8 * (c >> 1) + 2 * (lane & 3) + (c & 1);
      if ((lane >> 2) == 0 && row < R)
        a.buf.part_stats[((long long)z * a.buf.nsplit + blockIdx.x) * R + row] = make_float2(cm[c], cl[c]);
    }
  }
}

// Merge the per-split statistics (log2 domain): m = max_s m_s, l = sum_s l_s 2^(m_s - m); keep (m, 1/l).
__global__ void score_mma_combine_kernel(const float2* __restrict__ part, float2* __restrict__ stats,
                                         double* __restrict__ mu64, int nsplit, int R) {
  // one warp per query row, lanes over the splits
  pdl_wait();
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
    if (p.y > 0.f) l += (double)p.y * exp2((double)p.x - (double)m);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
  if (lane == 0) {
    stats[z * R + row] = make_float2(m, (float)(1.0 / l));
    if (mu64) mu64[z * R + row] = (double)m + log2(l);       // the same normaliser, unrounded, for the refinement
  }
}

}  // namespace

cudaError_t launch_score_combine_log2(const ScoreBuffers& buf, int nz, int R, cudaStream_t st) {
  const cudaError_t e = launch_pdl(score_mma_combine_kernel, dim3((R + 7) / 8, nz), dim3(256), 0, st,
                                   static_cast<const float2*>(buf.part_stats), buf.stats, buf.ref.mu64, buf.nsplit, R);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

bool score_mma_supported(int dtype, const Shape& s) {
  return dtype == SNAP_BF16 && s.d_qk == D && s.g * s.Lo <= 256;
}

// Candidate splits per (prompt, KV head) for the tensor-core score passes: about two waves of CTAs.
int score_mma_nsplit(const Shape& s, int n_scored, int max_le, int sm_count) {
  const int tiles = (max_le + TN - 1) / TN;
  const long long base = (long long)n_scored * s.Hkv;
  long long ns = (4LL * sm_count + base - 1) / base;
  if (ns > tiles) ns = tiles;
  if (ns > 256) ns = 256;
  if (ns < 1) ns = 1;
  return (int)ns;
}

cudaError_t launch_score_mma(const Shape& s, const SeqBatch& b, const void* q_obs, const KVSource& src,
                             const ScoreBuffers& buf, cudaStream_t st) {
  if (b.n_scored == 0) return cudaSuccess;
  MmaArgs a;
  a.q = static_cast<const __nv_bfloat16*>(q_obs);
  a.k = static_cast<const __nv_bfloat16*>(src.k);
  a.k_tok_b = src.k_tok_stride * 2; a.k_head_b = src.k_head_stride * 2;
  a.Hq = s.Hq; a.Hkv = s.Hkv; a.g = s.g; a.Lo = s.Lo; a.Ls = s.Ls; a.Lr = s.Lr;
  a.R = s.g * s.Lo; a.RP = (a.R + 31) / 32 * 32;
  a.scale_log2 = s.scale * 1.4426950408889634f;
  a.b = b; a.buf = buf;
  const int nrw = a.RP / 32;
  const size_t smem = (size_t)a.RP * ROW_B + 2 * KT_B + 2 * nrw * TN * sizeof(float);
  static SmemLimit limit1 = {}, limit2 = {};
  if (cudaError_t e = ensure_dyn_smem(score_mma_kernel<1>, 110 * 1024, limit1)) return e;
  if (cudaError_t e = ensure_dyn_smem(score_mma_kernel<2>, 110 * 1024, limit2)) return e;
  const int nz = b.n_scored * s.Hkv;
  dim3 grid(buf.nsplit, nz);
  if (!buf.ext_mu) {                                          // Eq. 4's normalisers, unless the caller has them
    score_mma_kernel<1><<<grid, 32 * nrw, smem, st>>>(a);
    count_launch();
    if (launch_score_combine_log2(buf, nz, a.R, st) != cudaSuccess) return cudaGetLastError();
  }
  score_mma_kernel<2><<<grid, 32 * nrw, smem, st>>>(a);
  count_launch();
  return cudaGetLastError();
}

}  // namespace snap
