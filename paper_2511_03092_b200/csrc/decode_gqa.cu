// Decode attention over the compressed cache (Section 3.3) for grouped-query bf16 layers with
// 128-wide heads -- the HBM-bound kernel of the decode step.
//
// Split-K flash decoding.  Grid = (splits, KV heads, sequences); a CTA of 4 warps streams its
// share of the valid cache rows ([0, min(len, Lsr)) then [Lsr, Lsr + valid_topk)) through a
// ring of shared-memory stages filled by bulk async copies (cp.async.bulk + mbarrier
// transaction counts; rows of one KV head are contiguous, so a tile is one or two copies per
// tensor).  K and V rows are each read from HBM exactly once.
//
// Per 64-row tile each warp owns 16 rows.  A half-warp covers one 256-byte row with 128-bit
// shared loads (lane = 8 dims); the lane-partial dot products of 8 rows x G heads are reduced
// with a transposing shuffle network (each step halves the values a lane holds), which costs
// ~4x fewer shuffles than reducing every dot product separately and leaves one row's logits in
// each lane.  Online softmax is per warp (running max in the log2 domain, per-lane partial
// sums), probabilities go through a small per-warp shared buffer and are re-read as broadcasts
// for the P.V accumulation, where a lane owns 8 output dims of all G heads.  Warps are merged
// once at the end; splits are merged by a second kernel, which also advances the sequence
// length when a token was appended.
//
// Fused append (Eq. 3): the CTA whose range contains the new token's slot stores the new K/V
// row to the cache and patches its staged tile, so the stale row is never used.
#include "snap_internal.cuh"

namespace snap {
namespace {

constexpr int D = 128, TILE = 64, NSTAGE = 3, NT = 128, NWARP = 4;
constexpr int ROW_B = D * 2, TILE_B = TILE * ROW_B, STAGE_B = 2 * TILE_B;
constexpr int PS = D + 2;                       // floats per partial: m, l, acc[D]
constexpr unsigned kWaitLimit = 1u << 22;       // bounded spin on an mbarrier

struct FastArgs {
  const __nv_bfloat16* q; const __nv_bfloat16* k_new; const __nv_bfloat16* v_new;
  const int* slot_ids;
  char* kc; char* vc;
  long long seq_b, head_b;                      // cache strides in bytes (K and V alike)
  int Hq, Hkv, Ls, Lr, max_seqs, nsplit;
  float scale_log2;                             // softmax_scale * log2(e)
  const int* seq_len; const int* valid_topk;
  float* partials;                              // [n_active][Hq][nsplit][PS]
  uint32_t* status;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Waits for the phase with the given parity; gives up after kWaitLimit polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, unsigned parity) {
  for (unsigned it = 0; it < kWaitLimit; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, unsigned bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// Rows [va, vb) of the valid-row index space -> one stage.  Index x < n_low is cache row x, the
// rest is row Lsr + (x - n_low): at most two contiguous pieces per tensor.
__device__ __forceinline__ void issue_tile(uint32_t stage, uint32_t bar, const char* kc, const char* vc,
                                           int va, int vb, int n_low, int Lsr) {
  mbar_expect_tx(bar, (unsigned)(vb - va) * ROW_B * 2);
  const int e1 = min(vb, n_low);
  if (va < e1) {
    const unsigned bytes = (unsigned)(e1 - va) * ROW_B;
    bulk_g2s(stage, kc + (long long)va * ROW_B, bytes, bar);
    bulk_g2s(stage + TILE_B, vc + (long long)va * ROW_B, bytes, bar);
  }
  const int s2 = max(va, n_low);
  if (s2 < vb) {
    const unsigned bytes = (unsigned)(vb - s2) * ROW_B, off = (unsigned)(s2 - va) * ROW_B;
    const long long src = (long long)(Lsr + s2 - n_low) * ROW_B;
    bulk_g2s(stage + off, kc + src, bytes, bar);
    bulk_g2s(stage + TILE_B + off, vc + src, bytes, bar);
  }
}

__device__ __forceinline__ void unpack8(const uint4& u, float (&f)[8]) {
  f[0] = __uint_as_float(u.x << 16); f[1] = __uint_as_float(u.x & 0xffff0000u);
  f[2] = __uint_as_float(u.y << 16); f[3] = __uint_as_float(u.y & 0xffff0000u);
  f[4] = __uint_as_float(u.z << 16); f[5] = __uint_as_float(u.z & 0xffff0000u);
  f[6] = __uint_as_float(u.w << 16); f[7] = __uint_as_float(u.w & 0xffff0000u);
}

template <int G>
__global__ void __launch_bounds__(NT, 2) decode_gqa_kernel(const FastArgs a) {
  constexpr int VPL = G / 2;                    // logits a lane holds after the reduction
  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char* stages = smem_raw;                                   // NSTAGE x (K tile | V tile)
  float* pbuf = reinterpret_cast<float*>(smem_raw + NSTAGE * STAGE_B);  // [NWARP][2][8][G]
  uint64_t* bars = reinterpret_cast<uint64_t*>(pbuf + NWARP * 16 * G);
  __shared__ int abort_flag;

  const int sp = blockIdx.x, kvh = blockIdx.y, i = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5, hw = lane >> 4, l16 = lane & 15;
  const int odd = l16 & 1, jrow = l16 >> 1;
  const int slot = a.slot_ids[i];
  const bool bad = slot < 0 || slot >= a.max_seqs;
  const int Lsr = a.Ls + a.Lr;
  int n_low = 0, n_valid = 0, new_slot = -1;
  if (!bad) {
    const int t = a.seq_len[slot];
    n_low = min(t + (a.k_new ? 1 : 0), Lsr);
    n_valid = n_low + a.valid_topk[slot];
    if (a.k_new) new_slot = ring_slot(t, a.Ls, a.Lr);
  } else if (tid == 0 && sp == 0 && kvh == 0 && a.status) {
    atomicOr(a.status, SNAP_DEV_BAD_SLOT);
  }
  // even split of the tiles of this (sequence, KV head) over the splits
  const int ntiles = (n_valid + TILE - 1) / TILE;
  const int t_begin = (int)((long long)ntiles * sp / a.nsplit);
  const int t_end = (int)((long long)ntiles * (sp + 1) / a.nsplit);
  const int v0 = t_begin * TILE, v1 = min(n_valid, t_end * TILE);
  const int T = t_end - t_begin;

  char* kc = a.kc + slot * a.seq_b + kvh * a.head_b;
  char* vc = a.vc + slot * a.seq_b + kvh * a.head_b;
  const __nv_bfloat16* kn = a.k_new ? a.k_new + ((long long)i * a.Hkv + kvh) * D : nullptr;
  const __nv_bfloat16* vn = a.v_new ? a.v_new + ((long long)i * a.Hkv + kvh) * D : nullptr;

  const uint32_t stage0 = smem_u32(stages), bar0 = smem_u32(bars);
  if (tid == 0) {
    abort_flag = 0;
    for (int s = 0; s < NSTAGE; ++s) mbar_init(bar0 + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (tid == 0) {
    for (int s = 0; s < NSTAGE && s < T; ++s)
      issue_tile(stage0 + s * STAGE_B, bar0 + 8 * s, kc, vc, v0 + s * TILE, min(v1, v0 + (s + 1) * TILE),
                 n_low, Lsr);
  }
  // the owner of the new token's slot stores it (its staged copy is patched below)
  const bool owns_new = new_slot >= v0 && new_slot < v1;
  if (owns_new && w == 0) {
    const uint4* srcp = reinterpret_cast<const uint4*>(hw == 0 ? kn : vn);
    char* dst = (hw == 0 ? kc : vc) + (long long)new_slot * ROW_B;
    reinterpret_cast<uint4*>(dst)[l16] = srcp[l16];
  }

  // query rows of the group, pre-scaled so that exp2 can be used directly
  float q[G][8];
  {
    const __nv_bfloat16* qp = a.q + ((long long)i * a.Hq + (long long)kvh * G) * D + l16 * 8;
#pragma unroll
    for (int h = 0; h < G; ++h) {
      const uint4 u = *reinterpret_cast<const uint4*>(qp + h * D);
      unpack8(u, q[h]);
#pragma unroll
      for (int c = 0; c < 8; ++c) q[h][c] *= a.scale_log2;
    }
  }
  float acc[G][8], m_run[G], l_lane[VPL];
#pragma unroll
  for (int h = 0; h < G; ++h) {
    m_run[h] = -INFINITY;
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[h][c] = 0.f;
  }
#pragma unroll
  for (int e = 0; e < VPL; ++e) l_lane[e] = 0.f;
  float* pw = pbuf + (w * 2 + hw) * 8 * G;      // this half-warp's probabilities [8][G]

  for (int t = 0; t < T; ++t) {
    const int s = t % NSTAGE;
    const unsigned parity = (unsigned)(t / NSTAGE) & 1u;
    if (!mbar_wait(bar0 + 8 * s, parity)) {
      abort_flag = 1;
      if (a.status) atomicOr(a.status, SNAP_DEV_WAIT_TIMEOUT);
    }
    const int va = v0 + t * TILE;
    const int nrows = min(TILE, v1 - va);
    unsigned char* sK = stages + s * STAGE_B;
    unsigned char* sV = sK + TILE_B;
    const bool patch = new_slot >= va && new_slot < va + nrows;
    if (patch || nrows < TILE) {                 // rare: new-token row, or the ragged last tile
      if (patch && w == 0) {
        const uint4* srcp = reinterpret_cast<const uint4*>(hw == 0 ? kn : vn);
        reinterpret_cast<uint4*>((hw == 0 ? sK : sV) + (new_slot - va) * ROW_B)[l16] = srcp[l16];
      }
      for (int e = tid; e < (TILE - nrows) * (ROW_B / 16); e += NT) {      // zero rows past the end
        reinterpret_cast<uint4*>(sK + nrows * ROW_B)[e] = make_uint4(0, 0, 0, 0);
        reinterpret_cast<uint4*>(sV + nrows * ROW_B)[e] = make_uint4(0, 0, 0, 0);
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncthreads();
    }

    // ---- logits: lane-partial dot products of 8 rows x G heads ----
    float part[8 * G];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int row = 16 * w + 2 * j + hw;
      const uint4 u = *reinterpret_cast<const uint4*>(sK + row * ROW_B + l16 * 16);
      float kf[8];
      unpack8(u, kf);
#pragma unroll
      for (int h = 0; h < G; ++h) {
        float sacc = q[h][0] * kf[0];
#pragma unroll
        for (int c = 1; c < 8; ++c) sacc = fmaf(q[h][c], kf[c], sacc);
        part[j * G + h] = sacc;
      }
    }
    // transposing reduction over the 16 lanes of a half-warp
#pragma unroll
    for (int bit = 8, width = 4 * G; bit >= 1; bit >>= 1, width >>= 1) {
      const bool upper = (lane & bit) != 0;
#pragma unroll
      for (int e = 0; e < width; ++e) {
        const float send = upper ? part[e] : part[e + width];
        const float keep = upper ? part[e + width] : part[e];
        part[e] = keep + __shfl_xor_sync(0xffffffffu, send, bit);
      }
    }
    // lane now holds row (16w + 2*jrow + hw), heads odd*VPL .. odd*VPL+VPL-1
    const bool row_ok = 16 * w + 2 * jrow + hw < nrows;
    float mx[VPL];
#pragma unroll
    for (int e = 0; e < VPL; ++e) {
      part[e] = row_ok ? part[e] : -INFINITY;
      mx[e] = part[e];
#pragma unroll
      for (int o = 2; o <= 16; o <<= 1) mx[e] = fmaxf(mx[e], __shfl_xor_sync(0xffffffffu, mx[e], o));
    }
    float m_use[G];
    bool changed = false;
#pragma unroll
    for (int e = 0; e < VPL; ++e) {
      const float other = __shfl_xor_sync(0xffffffffu, mx[e], 1);
      const float lo = odd ? other : mx[e], hi = odd ? mx[e] : other;
      const float n_lo = fmaxf(m_run[e], lo), n_hi = fmaxf(m_run[VPL + e], hi);
      changed |= (n_lo > m_run[e]) | (n_hi > m_run[VPL + e]);
      m_use[e] = n_lo; m_use[VPL + e] = n_hi;
    }
    if (changed) {                               // warp-uniform: every lane sees the same maxima
      float al[G];
#pragma unroll
      for (int h = 0; h < G; ++h) {
        al[h] = m_run[h] == -INFINITY ? 0.f : exp2f(m_run[h] - m_use[h]);
        m_run[h] = m_use[h];
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[h][c] *= al[h];
      }
#pragma unroll
      for (int e = 0; e < VPL; ++e) l_lane[e] *= odd ? al[VPL + e] : al[e];
    }
    float pv[VPL];
#pragma unroll
    for (int e = 0; e < VPL; ++e) {
      const float mh = odd ? m_run[VPL + e] : m_run[e];
      pv[e] = exp2f(part[e] - (mh == -INFINITY ? 0.f : mh));
      l_lane[e] += pv[e];
    }
    if (VPL == 2) {
      *reinterpret_cast<float2*>(pw + jrow * G + odd * VPL) = make_float2(pv[0], pv[VPL - 1]);
    } else {
#pragma unroll
      for (int e = 0; e < VPL; ++e) pw[jrow * G + odd * VPL + e] = pv[e];
    }
    __syncwarp();
    // ---- P.V: a lane owns 8 output dims of all G heads ----
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int row = 16 * w + 2 * j + hw;
      const uint4 u = *reinterpret_cast<const uint4*>(sV + row * ROW_B + l16 * 16);
      float vf[8];
      unpack8(u, vf);
      float pj[G];
      if (G == 4) {
        const float4 p4 = *reinterpret_cast<const float4*>(pw + j * G);
        pj[0] = p4.x; pj[1] = p4.y; pj[2] = p4.z; pj[G - 1] = p4.w;
      } else {
#pragma unroll
        for (int h = 0; h < G; ++h) pj[h] = pw[j * G + h];
      }
#pragma unroll
      for (int h = 0; h < G; ++h)
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[h][c] = fmaf(pj[h], vf[c], acc[h][c]);
    }
    __syncthreads();
    if (abort_flag) break;
    if (tid == 0 && t + NSTAGE < T) {
      const int nv = v0 + (t + NSTAGE) * TILE;
      issue_tile(stage0 + s * STAGE_B, bar0 + 8 * s, kc, vc, nv, min(v1, nv + TILE), n_low, Lsr);
    }
  }

  // ---- merge the two half-warps, then the four warps, and write the split's partial ----
#pragma unroll
  for (int h = 0; h < G; ++h)
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[h][c] += __shfl_xor_sync(0xffffffffu, acc[h][c], 16);
#pragma unroll
  for (int e = 0; e < VPL; ++e)
#pragma unroll
    for (int o = 2; o <= 16; o <<= 1) l_lane[e] += __shfl_xor_sync(0xffffffffu, l_lane[e], o);
  float* wm = reinterpret_cast<float*>(stages);            // [NWARP][G]
  float* wl = wm + NWARP * G;                              // [NWARP][G]
  float* wacc = wl + NWARP * G;                            // [NWARP][G][D]
  if (lane < 2) {
#pragma unroll
    for (int e = 0; e < VPL; ++e) {
      wm[w * G + lane * VPL + e] = lane ? m_run[VPL + e] : m_run[e];
      wl[w * G + lane * VPL + e] = l_lane[e];
    }
  }
  if (hw == 0) {
#pragma unroll
    for (int h = 0; h < G; ++h)
#pragma unroll
      for (int c = 0; c < 8; ++c) wacc[(w * G + h) * D + l16 * 8 + c] = acc[h][c];
  }
  __syncthreads();
  float* part_out = a.partials + (((long long)i * a.Hq + (long long)kvh * G) * a.nsplit + sp) * PS;
#pragma unroll
  for (int h = 0; h < G; ++h) {
    float M = -INFINITY;
#pragma unroll
    for (int ww = 0; ww < NWARP; ++ww) M = fmaxf(M, wm[ww * G + h]);
    float L = 0.f, O = 0.f;
#pragma unroll
    for (int ww = 0; ww < NWARP; ++ww) {
      const float mw = wm[ww * G + h];
      const float f = mw == -INFINITY ? 0.f : exp2f(mw - M);
      L += wl[ww * G + h] * f;
      O += wacc[(ww * G + h) * D + tid] * f;
    }
    float* ph = part_out + (long long)h * a.nsplit * PS;
    if (tid == 0) { ph[0] = M; ph[1] = L; }
    ph[2 + tid] = O;
  }
}

// Merge the splits of one (sequence, query head); maxima are in the log2 domain.
__global__ void __launch_bounds__(D) decode_gqa_merge_kernel(const float* __restrict__ partials,
                                                             __nv_bfloat16* __restrict__ out, int Hq,
                                                             int nsplit, const int* __restrict__ slot_ids,
                                                             int* seq_len, int max_seqs, int bump) {
  const int h = blockIdx.x, i = blockIdx.y, t = threadIdx.x;
  const float* p = partials + ((long long)i * Hq + h) * nsplit * PS;
  float M = -INFINITY;
  for (int s = 0; s < nsplit; ++s) M = fmaxf(M, p[s * PS]);
  float L = 0.f, O = 0.f;
  for (int s = 0; s < nsplit; ++s) {
    const float ms = p[s * PS];
    const float f = ms == -INFINITY ? 0.f : exp2f(ms - M);
    L += p[s * PS + 1] * f;
    O += p[s * PS + 2 + t] * f;
  }
  out[((long long)i * Hq + h) * D + t] = __float2bfloat16_rn(L > 0.f ? O / L : 0.f);
  if (bump && h == 0 && t == 0) {
    const int slot = slot_ids[i];
    if (slot >= 0 && slot < max_seqs) seq_len[slot] += 1;
  }
}

template <int G>
cudaError_t launch_g(const FastArgs& a, int n_active, __nv_bfloat16* out, int* seq_len, int bump,
                     cudaStream_t st) {
  const size_t smem = (size_t)NSTAGE * STAGE_B + NWARP * 16 * G * sizeof(float) + NSTAGE * 8;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(decode_gqa_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  dim3 grid(a.nsplit, a.Hkv, n_active);
  decode_gqa_kernel<G><<<grid, NT, smem, st>>>(a);
  count_launch();
  dim3 mgrid(a.Hq, n_active);
  decode_gqa_merge_kernel<<<mgrid, D, 0, st>>>(a.partials, out, a.Hq, a.nsplit, a.slot_ids, seq_len,
                                               a.max_seqs, bump);
  count_launch();
  return cudaGetLastError();
}

}  // namespace

bool decode_gqa_supported(int dtype, const Shape& s) {
  return dtype == SNAP_BF16 && s.d_qk == D && s.d_v == D && !s.v_aliases_k && (s.g == 2 || s.g == 4 || s.g == 8);
}

// Splits per (sequence, KV head): enough CTAs to fill two per SM, preferring counts whose last
// wave is nearly full, with at least one tile per split.
int decode_gqa_nsplit(const Shape& s, int n_active, int sm_count) {
  const int tiles = (s.Sc + TILE - 1) / TILE;
  const long long base = (long long)n_active * s.Hkv;
  const double slots = 2.0 * sm_count;
  int best = 1;
  double best_score = -1.0;
  const int max_ns = tiles < 64 ? tiles : 64;
  for (int ns = 1; ns <= max_ns; ++ns) {
    const double waves = base * ns / slots;
    const double full = waves < 1.0 ? waves : waves / (double)(long long)(waves + 0.999999);
    const double per_split = (double)tiles / ns;
    const double overhead = per_split / (per_split + 1.5);      // pipeline fill and merge per split
    const double score = full * overhead;
    if (score > best_score + 1e-9) { best_score = score; best = ns; }
  }
  return best;
}

size_t decode_gqa_partial_floats(const Shape& s, int n_active, int nsplit) {
  return (size_t)n_active * s.Hq * nsplit * PS;
}

cudaError_t launch_decode_gqa(const Shape& s, const void* q, const void* k_new, const void* v_new,
                              const int* slot_ids, int n_active, void* k_cache, void* v_cache,
                              int* seq_len, const int* valid_topk, void* out, float* partials,
                              int nsplit, uint32_t* status, cudaStream_t st) {
  if (n_active == 0) return cudaSuccess;
  FastArgs a;
  a.q = static_cast<const __nv_bfloat16*>(q);
  a.k_new = static_cast<const __nv_bfloat16*>(k_new);
  a.v_new = static_cast<const __nv_bfloat16*>(v_new);
  a.slot_ids = slot_ids;
  a.kc = static_cast<char*>(k_cache); a.vc = static_cast<char*>(v_cache);
  a.head_b = (long long)s.Sc * ROW_B; a.seq_b = a.head_b * s.Hkv;
  a.Hq = s.Hq; a.Hkv = s.Hkv; a.Ls = s.Ls; a.Lr = s.Lr; a.max_seqs = s.max_seqs; a.nsplit = nsplit;
  a.scale_log2 = s.scale * 1.4426950408889634f;
  a.seq_len = seq_len; a.valid_topk = valid_topk; a.partials = partials; a.status = status;
  __nv_bfloat16* o = static_cast<__nv_bfloat16*>(out);
  const int bump = k_new != nullptr;
  switch (s.g) {
    case 2: return launch_g<2>(a, n_active, o, seq_len, bump, st);
    case 4: return launch_g<4>(a, n_active, o, seq_len, bump, st);
    case 8: return launch_g<8>(a, n_active, o, seq_len, bump, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace snap
