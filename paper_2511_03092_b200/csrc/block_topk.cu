// Per-step block top-K over the prompt's middle -- the alternative to a one-time top-K that the
// paper's related-work section leaves to future work (KV blocks with pre-computed statistics, the
// top ones looked up for every decoded token).
//
// The middle of the prompt is kept whole, in position order, in the third section of a cache whose
// top-K budget is at least the prompt's middle (snap_compress then keeps every candidate).  Two
// kernels here, for bf16 caches:
//   block_stats_kernel   once per prompt: element-wise minimum and maximum of the keys of every block of
//                        `block_tokens` consecutive rows of that section (the last block may be
//                        shorter), per KV head: stats[slot][kvh][block][0 = min, 1 = max][d_qk].
//   block_score_kernel   every step: block b of KV head kvh scores
//                            U = sum over the group's heads h, dims d of max(q[h][d] * min[d], q[h][d] * max[d]),
//                        an upper bound of the group-summed logit of every key of the block.  Since
//                        min <= max, the larger product is q * max for q >= 0 and q * min otherwise, so
//                        U = max . Q+ + min . Q- with Q+[d] = sum_h max(q[h][d], 0), Q-[d] = sum_h min(q[h][d], 0):
//                        one pass over the statistics (512 bytes per block at d = 128), a warp-wide
//                        16-byte load per block, in single precision; next to U the kernel writes
//                        A = sum of the absolute values of U's terms, which bounds U's rounding error.
//   block_select_kernel  the n_blocks highest-scoring blocks of each (sequence, KV head), listed in
//                        ascending order, ties to the lower index: four 8-bit radix passes over the
//                        order-preserving integer images of the scores find the threshold; the blocks
//                        whose single-precision score cannot be told from the threshold (within
//                        2e-5 (A + A_threshold)) are scored again in double precision -- a few
//                        blocks, 256 multiply-adds each -- and ranked by that, so the selection is
//                        the one the exact scores give (down to 1e-15 relative); then an ordered
//                        emission.  More than 256 such blocks: the single-precision order stands
//                        and SNAP_DEV_BAND_OVERFLOW is raised.
// The decode kernel then visits the listed blocks instead of the whole section (decode_gqa_mma.cu).
#include "snap_internal.cuh"

namespace snap {
namespace {

constexpr int SEL_NT = 256, MAX_BLOCKS = 8192;

struct StatsArgs {
  const __nv_bfloat16* kc;      // cache keys [max_seqs][Hkv][Sc][d]
  __nv_bfloat16* stats;         // [max_seqs][Hkv][nb_max][2][d]
  const int* slot_ids; const int* valid_topk;
  int Hkv, d, Sc, Lsr, max_seqs, nb_max, bs;
  uint32_t* status;
};

// grid (nb_max, Hkv, n), d / 2 threads: thread = two adjacent dims.
__global__ void block_stats_kernel(const StatsArgs a) {
  const int b = blockIdx.x, kvh = blockIdx.y, i = blockIdx.z;
  const int slot = a.slot_ids[i];
  if (slot < 0 || slot >= a.max_seqs) {
    if (threadIdx.x == 0 && b == 0 && kvh == 0 && a.status) atomicOr(a.status, SNAP_DEV_BAD_SLOT);
    return;
  }
  const int n_top = a.valid_topk[slot];
  const int r0 = b * a.bs, r1 = min(r0 + a.bs, n_top);
  if (r0 >= r1) return;                                        // no such block for this prompt
  const __nv_bfloat16* rows = a.kc + (((long long)slot * a.Hkv + kvh) * a.Sc + a.Lsr) * a.d;
  const int c = 2 * threadIdx.x;
  __nv_bfloat162 mn = *reinterpret_cast<const __nv_bfloat162*>(rows + (long long)r0 * a.d + c), mx = mn;
  for (int r = r0 + 1; r < r1; ++r) {
    const __nv_bfloat162 v = *reinterpret_cast<const __nv_bfloat162*>(rows + (long long)r * a.d + c);
    mn = __hmin2(mn, v);
    mx = __hmax2(mx, v);
  }
  __nv_bfloat16* out = a.stats + ((((long long)slot * a.Hkv + kvh) * a.nb_max + b) * 2) * a.d;
  *reinterpret_cast<__nv_bfloat162*>(out + c) = mn;
  *reinterpret_cast<__nv_bfloat162*>(out + a.d + c) = mx;
}

struct SelectArgs {
  const __nv_bfloat16* q;       // [n_active][Hq][d]
  const __nv_bfloat16* stats;
  const int* slot_ids; const int* valid_topk;
  uint2* keys;                  // scratch [n_active][Hkv][nb_max]: (order-preserving integer image of U, bits of A)
  int* block_idx;               // [n_active][Hkv][n_blocks]
  int* n_sel;                   // [n_active][Hkv]
  int Hq, Hkv, g, d, max_seqs, nb_max, bs, n_blocks;
  int no_rescoring;             // testing aid (option SNAP_OPT_REFINE_OFF): keep the single-precision order
  uint32_t* status;
};

// order-preserving map of a float to an unsigned key (larger float = larger key)
__device__ __forceinline__ unsigned key_of(float x) {
  const unsigned u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// grid (ceil(nb_max / 256), Hkv, n_active), 256 threads: a warp takes 32 blocks, four at a time; a lane owns the same
// 16-byte chunk (eight dims of the minimum row, or of the maximum row) of every block it visits.
constexpr int SC_BLOCKS = 256, SC_PER_WARP = SC_BLOCKS / 8;
__global__ void __launch_bounds__(256) block_score_kernel(const SelectArgs a) {
  const int kvh = blockIdx.y, i = blockIdx.z, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int slot = a.slot_ids[i];
  if (slot < 0 || slot >= a.max_seqs) return;                  // the selection kernel reports it
  const int nb = min((a.valid_topk[slot] + a.bs - 1) / a.bs, a.nb_max);
  const int b_first = blockIdx.x * SC_BLOCKS + warp * SC_PER_WARP;
  if (b_first >= nb) return;
  const int cpr = a.d / 8, cpb = 2 * cpr;                      // 16-byte chunks per row and per block (min row, max row)
  // this lane's chunks: lane, lane + 32 (d = 256); per chunk eight entries of Q- (minimum row) or Q+ (maximum row)
  float w[2][8];
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    const int c = lane + 32 * t;
#pragma unroll
    for (int e = 0; e < 8; ++e) w[t][e] = 0.f;
    if (c < cpb) {
      const bool is_max = c >= cpr;
      const int d0 = (is_max ? c - cpr : c) * 8;
      for (int h = 0; h < a.g; ++h) {
        const uint4 raw = *reinterpret_cast<const uint4*>(a.q + ((long long)i * a.Hq + (long long)kvh * a.g + h) * a.d + d0);
        const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 f = __bfloat1622float2(p2[e]);
          w[t][2 * e] += is_max ? fmaxf(f.x, 0.f) : fminf(f.x, 0.f);
          w[t][2 * e + 1] += is_max ? fmaxf(f.y, 0.f) : fminf(f.y, 0.f);
        }
      }
    }
  }
  const uint4* st = reinterpret_cast<const uint4*>(a.stats + (((long long)slot * a.Hkv + kvh) * a.nb_max) * 2 * a.d);
  uint2* out = a.keys + ((long long)i * a.Hkv + kvh) * a.nb_max;
#pragma unroll 1
  for (int b0 = b_first; b0 < min(b_first + SC_PER_WARP, nb); b0 += 4) {
    uint4 v[4][2];
#pragma unroll
    for (int k = 0; k < 4; ++k)
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        const int c = lane + 32 * t;
        v[k][t] = b0 + k < nb && c < cpb ? st[(long long)(b0 + k) * cpb + c] : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      float u = 0.f, ab = 0.f;
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&v[k][t]);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 f = __bfloat1622float2(p2[e]);
          u = fmaf(f.x, w[t][2 * e], u);
          u = fmaf(f.y, w[t][2 * e + 1], u);
          ab = fmaf(fabsf(f.x), fabsf(w[t][2 * e]), ab);
          ab = fmaf(fabsf(f.y), fabsf(w[t][2 * e + 1]), ab);
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        u += __shfl_xor_sync(0xffffffffu, u, o);
        ab += __shfl_xor_sync(0xffffffffu, ab, o);
      }
      if (lane == 0 && b0 + k < nb) out[b0 + k] = make_uint2(key_of(u), __float_as_uint(ab));
    }
  }
}

// Block-wide exclusive scan of one int per thread (SEL_NT threads); returns the exclusive prefix and the total.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_tot, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) { const int u = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += u; }
  __syncthreads();                                             // warp_tot may still be read from the previous scan
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  int before = 0, tot = 0;
#pragma unroll
  for (int w2 = 0; w2 < SEL_NT / 32; ++w2) { const int t = warp_tot[w2]; tot += t; if (w2 < warp) before += t; }
  total = tot;
  return before + incl - v;
}

__device__ __forceinline__ float float_of_key(unsigned k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

constexpr int BAND_CAP = 256;
constexpr float BAND_REL = 2e-5f;      // 256 single-precision multiply-adds: |error| <= 256 * 2^-24 * A = 1.5e-5 A

// grid (Hkv, n_active), SEL_NT threads.  Dynamic shared memory: keys [nb] | take flags [nb].
__global__ void __launch_bounds__(SEL_NT) block_select_kernel(const SelectArgs a) {
  extern __shared__ unsigned char sel_smem[];
  unsigned* keys = reinterpret_cast<unsigned*>(sel_smem);             // [nb]
  unsigned char* take = reinterpret_cast<unsigned char*>(keys + a.nb_max);   // [nb]
  __shared__ int hist[256], warp_tot[SEL_NT / 32];
  __shared__ unsigned s_prefix;
  __shared__ int s_need, s_nband, s_nsure, s_thr_block;
  __shared__ int band_idx[BAND_CAP];
  __shared__ double band_u[BAND_CAP];
  const int kvh = blockIdx.x, i = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int slot = a.slot_ids[i];
  int* out = a.block_idx + ((long long)i * a.Hkv + kvh) * a.n_blocks;
  if (slot < 0 || slot >= a.max_seqs) {
    if (tid == 0) {
      a.n_sel[i * a.Hkv + kvh] = 0;
      if (kvh == 0 && a.status) atomicOr(a.status, SNAP_DEV_BAD_SLOT);
    }
    return;
  }
  const int n_top = a.valid_topk[slot];
  const int nb = min((n_top + a.bs - 1) / a.bs, a.nb_max);
  const int want = min(a.n_blocks, nb);
  if (want == nb) {                                            // every block: no selection needed
    for (int b = tid; b < nb; b += SEL_NT) out[b] = b;
    if (tid == 0) a.n_sel[i * a.Hkv + kvh] = nb;
    return;
  }
  const uint2* scored = a.keys + ((long long)i * a.Hkv + kvh) * a.nb_max;
  for (int b = tid; b < nb; b += SEL_NT) keys[b] = scored[b].x;
  if (tid == 0) { s_nband = 0; s_nsure = 0; s_thr_block = 0x7fffffff; }
  // ---- the want-th largest single-precision score by four 8-bit radix passes ----
  unsigned prefix = 0u;
  int need = want;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    hist[tid] = 0;                                             // SEL_NT == 256 bins
    __syncthreads();
    const unsigned himask = pass == 0 ? 0u : 0xffffffffu << (shift + 8);
    for (int b = tid; b < nb; b += SEL_NT) {
      const unsigned k = keys[b];
      if ((k & himask) == prefix) atomicAdd(&hist[(k >> shift) & 255u], 1);
    }
    __syncthreads();
    // thread t looks at digit 255 - t: `above` = keys (under the prefix) with a larger digit
    int total;
    const int mine = hist[255 - tid];
    const int above = block_exclusive_scan(mine, warp_tot, total);
    if (above < need && above + mine >= need) {               // exactly one thread: the digit of the want-th largest key
      s_prefix = prefix | ((unsigned)(255 - tid) << shift);
      s_need = need - above;
    }
    __syncthreads();
    prefix = s_prefix;
    need = s_need;                                             // how many of the keys equal so far are still wanted
  }
  const unsigned tau = prefix;
  const int need_eq = need;                                    // single-precision rule: this many of the blocks at the threshold
  // ---- which blocks can single precision not tell from the threshold? ----
  for (int b = tid; b < nb; b += SEL_NT)
    if (keys[b] == tau) atomicMin(&s_thr_block, b);
  __syncthreads();
  const float tau_f = float_of_key(tau), a_tau = __uint_as_float(scored[s_thr_block].y);
  for (int b = tid; b < nb; b += SEL_NT) {
    const float u = float_of_key(keys[b]);
    const float band = BAND_REL * (__uint_as_float(scored[b].y) + a_tau);
    unsigned char t = 0;
    if (u - tau_f > band) { t = 1; atomicAdd(&s_nsure, 1); }   // above the threshold whatever the rounding
    else if (tau_f - u <= band) {                              // undecided
      const int m = atomicAdd(&s_nband, 1);
      if (m < BAND_CAP) band_idx[m] = b;
    }
    take[b] = t;
  }
  __syncthreads();
  const int n_band = s_nband, n_sure = s_nsure;
  if (n_band <= BAND_CAP && !a.no_rescoring) {
    // ---- their scores again, in double precision: a warp per block, a lane per 16-byte chunk ----
    const int cpr = a.d / 8, cpb = 2 * cpr;
    if (warp < n_band) {
      double w[2][8];
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        const int c = lane + 32 * t;
#pragma unroll
        for (int e = 0; e < 8; ++e) w[t][e] = 0.0;
        if (c < cpb) {
          const bool is_max = c >= cpr;
          const int d0 = (is_max ? c - cpr : c) * 8;
          for (int h = 0; h < a.g; ++h) {
            const uint4 raw = *reinterpret_cast<const uint4*>(a.q + ((long long)i * a.Hq + (long long)kvh * a.g + h) * a.d + d0);
            const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float2 f = __bfloat1622float2(p2[e]);
              w[t][2 * e] += (double)(is_max ? fmaxf(f.x, 0.f) : fminf(f.x, 0.f));
              w[t][2 * e + 1] += (double)(is_max ? fmaxf(f.y, 0.f) : fminf(f.y, 0.f));
            }
          }
        }
      }
      const uint4* st = reinterpret_cast<const uint4*>(a.stats + (((long long)slot * a.Hkv + kvh) * a.nb_max) * 2 * a.d);
      for (int m = warp; m < n_band; m += SEL_NT / 32) {
        double u = 0.0;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          const int c = lane + 32 * t;
          if (c < cpb) {
            const uint4 v = st[(long long)band_idx[m] * cpb + c];
            const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float2 f = __bfloat1622float2(p2[e]);
              u = fma((double)f.x, w[t][2 * e], u);
              u = fma((double)f.y, w[t][2 * e + 1], u);
            }
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) u += __shfl_xor_sync(0xffffffffu, u, o);
        if (lane == 0) band_u[m] = u;
      }
    }
    __syncthreads();
    // ---- the best (want - n_sure) of them: larger score first, lower block number on equal scores ----
    const int room = want - n_sure;
    for (int m = tid; m < n_band; m += SEL_NT) {
      const double um = band_u[m];
      const int bm = band_idx[m];
      int rank = 0;
      for (int o = 0; o < n_band; ++o) rank += band_u[o] > um || (band_u[o] == um && band_idx[o] < bm);
      if (rank < room) take[bm] = 1;
    }
  } else {
    // too many to re-score: the single-precision order stands (blocks at the threshold by block number)
    if (tid == 0 && a.status && !a.no_rescoring) atomicOr(a.status, SNAP_DEV_BAND_OVERFLOW);
    const int run0 = (nb + SEL_NT - 1) / SEL_NT, c0 = tid * run0, c1 = min(c0 + run0, nb);
    int n_eq = 0;
    for (int b = c0; b < c1; ++b) n_eq += keys[b] == tau;
    int total;
    int eq_rank = block_exclusive_scan(n_eq, warp_tot, total);
    for (int b = c0; b < c1; ++b) {
      const unsigned k = keys[b];
      take[b] = k > tau || (k == tau && eq_rank < need_eq);
      eq_rank += k == tau;
    }
  }
  __syncthreads();
  // ---- ordered emission: a thread owns a run of consecutive blocks ----
  const int run = (nb + SEL_NT - 1) / SEL_NT, b0 = tid * run, b1 = min(b0 + run, nb);
  int n_take = 0;
  for (int b = b0; b < b1; ++b) n_take += take[b];
  int total;
  int pos = block_exclusive_scan(n_take, warp_tot, total);
  for (int b = b0; b < b1; ++b)
    if (take[b] && pos < want) out[pos++] = b;
  if (tid == 0) a.n_sel[i * a.Hkv + kvh] = want;
}

}  // namespace

int block_count_max(const Shape& s, int block_tokens) { return (s.K + block_tokens - 1) / block_tokens; }

bool block_topk_supported(int dtype, const Shape& s, int block_tokens) {
  return dtype == SNAP_BF16 && !s.v_aliases_k && s.d_qk % 8 == 0 && s.d_qk <= 256 && block_tokens >= 16 && block_tokens % 16 == 0 &&
         block_tokens <= 1024 && s.K > 0 && block_count_max(s, block_tokens) <= MAX_BLOCKS && s.g <= 16;
}

cudaError_t launch_block_stats(const Shape& s, int block_tokens, const int* slot_ids, int n, const void* k_cache,
                               const int* valid_topk, void* stats, uint32_t* status, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  StatsArgs a;
  a.kc = static_cast<const __nv_bfloat16*>(k_cache);
  a.stats = static_cast<__nv_bfloat16*>(stats);
  a.slot_ids = slot_ids; a.valid_topk = valid_topk;
  a.Hkv = s.Hkv; a.d = s.d_qk; a.Sc = s.Sc; a.Lsr = s.Ls + s.Lr; a.max_seqs = s.max_seqs;
  a.nb_max = block_count_max(s, block_tokens); a.bs = block_tokens; a.status = status;
  block_stats_kernel<<<dim3(a.nb_max, s.Hkv, n), s.d_qk / 2, 0, st>>>(a);
  count_launch();
  return cudaGetLastError();
}

size_t block_select_scratch_bytes(const Shape& s, int block_tokens, int n_active) {
  return (size_t)n_active * s.Hkv * block_count_max(s, block_tokens) * sizeof(uint2);
}

cudaError_t launch_block_select(const Shape& s, int block_tokens, int n_blocks, const void* q, const int* slot_ids,
                                int n_active, const void* stats, const int* valid_topk, int* block_idx, int* n_sel,
                                void* scratch, uint32_t* status, cudaStream_t st) {
  if (n_active == 0) return cudaSuccess;
  SelectArgs a;
  a.q = static_cast<const __nv_bfloat16*>(q);
  a.stats = static_cast<const __nv_bfloat16*>(stats);
  a.slot_ids = slot_ids; a.valid_topk = valid_topk; a.block_idx = block_idx; a.n_sel = n_sel;
  a.keys = static_cast<uint2*>(scratch);
  a.Hq = s.Hq; a.Hkv = s.Hkv; a.g = s.g; a.d = s.d_qk; a.max_seqs = s.max_seqs;
  a.nb_max = block_count_max(s, block_tokens); a.bs = block_tokens; a.n_blocks = n_blocks; a.status = status;
  a.no_rescoring = option(SNAP_OPT_REFINE_OFF) != 0;
  cudaError_t e = launch_pdl(block_score_kernel, dim3((a.nb_max + SC_BLOCKS - 1) / SC_BLOCKS, s.Hkv, n_active), dim3(256), 0, st, a);
  count_launch();
  if (e != cudaSuccess) return e;
  const size_t smem = (size_t)a.nb_max * (sizeof(unsigned) + 1) + 16;
  e = launch_pdl(block_select_kernel, dim3(s.Hkv, n_active), dim3(SEL_NT), smem, st, a);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace snap
