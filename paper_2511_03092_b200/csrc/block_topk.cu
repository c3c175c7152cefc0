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
//   block_select_kernel  every step: block b of KV head kvh scores
//                            U = sum over the group's heads h, dims d of max(q[h][d] * min[d], q[h][d] * max[d]),
//                        an upper bound of the group-summed logit of every key of the block; the
//                        n_blocks highest-scoring blocks are listed in ascending order, ties to
//                        the lower index.  The products of two bf16 values are exact in single
//                        precision; only the summation order rounds.
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
  int* block_idx;               // [n_active][Hkv][n_blocks]
  int* n_sel;                   // [n_active][Hkv]
  int Hq, Hkv, g, d, max_seqs, nb_max, bs, n_blocks;
  uint32_t* status;
};

// order-preserving map of a float to an unsigned key (larger float = larger key)
__device__ __forceinline__ unsigned key_of(float x) {
  const unsigned u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// grid (Hkv, n_active), SEL_NT threads.  Dynamic shared memory: q group as floats [g][d], keys [nb].
__global__ void __launch_bounds__(SEL_NT) block_select_kernel(const SelectArgs a) {
  extern __shared__ unsigned char sel_smem[];
  float* qs = reinterpret_cast<float*>(sel_smem);                     // [g][d]
  unsigned* keys = reinterpret_cast<unsigned*>(qs + a.g * a.d);       // [nb]
  __shared__ int hist[256];
  __shared__ unsigned s_prefix;
  __shared__ int s_need, s_warp_tot[SEL_NT / 32][2], s_run[2];
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
  for (int e = tid; e < a.g * a.d; e += SEL_NT)
    qs[e] = __bfloat162float(a.q[((long long)i * a.Hq + (long long)kvh * a.g) * a.d + e]);
  __syncthreads();
  // ---- scores: one warp per block, lanes over pairs of dims ----
  const __nv_bfloat16* st = a.stats + (((long long)slot * a.Hkv + kvh) * a.nb_max) * 2 * a.d;
  for (int b = warp; b < nb; b += SEL_NT / 32) {
    const __nv_bfloat16* mn = st + (long long)b * 2 * a.d, *mx = mn + a.d;
    float u = 0.f;
    for (int c = 2 * lane; c < a.d; c += 64) {
      const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(mn + c));
      const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(mx + c));
      for (int h = 0; h < a.g; ++h) {
        const float q0 = qs[h * a.d + c], q1 = qs[h * a.d + c + 1];
        u += fmaxf(q0 * lo.x, q0 * hi.x) + fmaxf(q1 * lo.y, q1 * hi.y);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) u += __shfl_xor_sync(0xffffffffu, u, o);
    if (lane == 0) keys[b] = key_of(u);
  }
  __syncthreads();
  if (want == nb) {                                            // every block: no selection needed
    for (int b = tid; b < nb; b += SEL_NT) out[b] = b;
    if (tid == 0) a.n_sel[i * a.Hkv + kvh] = nb;
    return;
  }
  // ---- the want-th largest key by four 8-bit radix passes ----
  if (tid == 0) { s_prefix = 0u; s_need = want; }
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    hist[tid] = 0;                                             // SEL_NT == 256 bins
    __syncthreads();
    const unsigned prefix = s_prefix, himask = pass == 0 ? 0u : 0xffffffffu << (shift + 8);
    for (int b = tid; b < nb; b += SEL_NT) {
      const unsigned k = keys[b];
      if ((k & himask) == prefix) atomicAdd(&hist[(k >> shift) & 255u], 1);
    }
    __syncthreads();
    if (tid == 0) {
      int need = s_need, digit = 255;
      for (; digit > 0; --digit) {                             // from the largest digit down
        if (hist[digit] >= need) break;
        need -= hist[digit];
      }
      s_prefix = prefix | ((unsigned)digit << shift);
      s_need = need;                                           // how many of the keys equal so far are still wanted
    }
    __syncthreads();
  }
  const unsigned tau = s_prefix;
  const int need_eq = s_need;                                  // blocks with key == tau to take, lowest indices first
  // ---- ordered emission: key > tau, and the first need_eq with key == tau ----
  if (tid == 0) { s_run[0] = 0; s_run[1] = 0; }                // blocks emitted, equal keys seen
  __syncthreads();
  for (int base = 0; base < nb; base += SEL_NT) {
    const int b = base + tid;
    const unsigned k = b < nb ? keys[b] : 0u;
    const int gt = b < nb && k > tau, eq = b < nb && k == tau;
    // exclusive scans of eq (to rank the equal keys) and of the emitted flags over the chunk
    int eq_incl = eq;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, eq_incl, o); if (lane >= o) eq_incl += v; }
    if (lane == 31) s_warp_tot[warp][1] = eq_incl;
    __syncthreads();
    int eq_before = s_run[1];
    for (int w2 = 0; w2 < warp; ++w2) eq_before += s_warp_tot[w2][1];
    const int take = gt || (eq && eq_before + eq_incl - 1 < need_eq);
    int tk_incl = take;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, tk_incl, o); if (lane >= o) tk_incl += v; }
    if (lane == 31) s_warp_tot[warp][0] = tk_incl;
    __syncthreads();
    int pos = s_run[0];
    for (int w2 = 0; w2 < warp; ++w2) pos += s_warp_tot[w2][0];
    if (take && pos + tk_incl - 1 < want) out[pos + tk_incl - 1] = b;
    __syncthreads();
    if (tid == 0) {
      int t0 = 0, t1 = 0;
      for (int w2 = 0; w2 < SEL_NT / 32; ++w2) { t0 += s_warp_tot[w2][0]; t1 += s_warp_tot[w2][1]; }
      s_run[0] += t0; s_run[1] += t1;
    }
    __syncthreads();
  }
  if (tid == 0) a.n_sel[i * a.Hkv + kvh] = want;
}

}  // namespace

int block_count_max(const Shape& s, int block_tokens) { return (s.K + block_tokens - 1) / block_tokens; }

bool block_topk_supported(int dtype, const Shape& s, int block_tokens) {
  return dtype == SNAP_BF16 && !s.v_aliases_k && s.d_qk % 2 == 0 && s.d_qk <= 512 && block_tokens >= 16 && block_tokens % 16 == 0 &&
         block_tokens <= 1024 && s.K > 0 && block_count_max(s, block_tokens) <= MAX_BLOCKS && s.g <= 8;
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

cudaError_t launch_block_select(const Shape& s, int block_tokens, int n_blocks, const void* q, const int* slot_ids,
                                int n_active, const void* stats, const int* valid_topk, int* block_idx, int* n_sel,
                                uint32_t* status, cudaStream_t st) {
  if (n_active == 0) return cudaSuccess;
  SelectArgs a;
  a.q = static_cast<const __nv_bfloat16*>(q);
  a.stats = static_cast<const __nv_bfloat16*>(stats);
  a.slot_ids = slot_ids; a.valid_topk = valid_topk; a.block_idx = block_idx; a.n_sel = n_sel;
  a.Hq = s.Hq; a.Hkv = s.Hkv; a.g = s.g; a.d = s.d_qk; a.max_seqs = s.max_seqs;
  a.nb_max = block_count_max(s, block_tokens); a.bs = block_tokens; a.n_blocks = n_blocks; a.status = status;
  const size_t smem = (size_t)s.g * s.d_qk * sizeof(float) + (size_t)a.nb_max * sizeof(unsigned);
  static SmemLimit limit = {};
  if (smem > 48 * 1024)
    if (cudaError_t e = ensure_dyn_smem(block_select_kernel, smem, limit)) return e;
  cudaError_t e = launch_pdl(block_select_kernel, dim3(s.Hkv, n_active), dim3(SEL_NT), smem, st, a);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace snap
