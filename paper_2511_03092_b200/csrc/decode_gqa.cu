// Decode attention over the compressed cache (Section 3.3) for bf16 layers with 128-wide heads
// and 1 to 8 query heads per KV head -- the HBM-bound kernel of the decode step.
//
// Split-K flash decoding.  Grid = (splits, KV heads, sequences).  A CTA's share of the valid
// cache rows ([0, min(len, Lsr)) then [Lsr, Lsr + valid_topk)) is cut into 16-row tiles that
// are dealt round-robin to its warps.  Every warp runs its own pipeline: a private ring of
// shared-memory stages filled by bulk async copies (cp.async.bulk completing on the warp's own
// mbarriers; the rows of one KV head are contiguous, so a tile is one or two copies per
// tensor), with no CTA-wide barrier in the loop.  K and V rows are read from HBM exactly once.
//
// Within a tile a half-warp covers one 256-byte row with 128-bit shared loads (lane = 8 dims).
// The lane-partial dot products of 8 rows x G heads are reduced with a transposing shuffle
// network (each step halves the values a lane holds), which needs ~4x fewer shuffles than
// reducing each dot product on its own and leaves one row's logits in each lane.  Online
// softmax is per warp (running max in the log2 domain, per-lane partial sums); probabilities
// go through a small per-half-warp shared buffer and come back as broadcasts for the P.V
// accumulation, where a lane owns 8 output dims of all G heads.  All multiply-adds are packed
// two-wide (fma.rn.f32x2), halving the issue slots of the arithmetic.  Warps are merged once at
// the end; splits are merged by a second kernel, which also advances the sequence length when
// a token was appended.
//
// Fused append (Eq. 3): the CTA whose range contains the new token's slot stores the new K/V
// row to the cache, and the warp that stages that row patches its copy, so the stale row is
// never used.
#include <cstdlib>

#include "snap_internal.cuh"

namespace snap {
namespace {

typedef unsigned long long u64;

constexpr int D = 128, WT = 16, NSTAGE = 2, NWARP = 4, NT = NWARP * 32;
constexpr int ROW_B = D * 2, WT_B = WT * ROW_B, STAGE_B = 2 * WT_B;   // stage = K tile | V tile
constexpr int PS = D + 2;                       // floats per partial: m, l, acc[D]
constexpr unsigned kWaitLimit = 1u << 22;       // bounded spin on an mbarrier

struct FastArgs {
  const __nv_bfloat16* q; const __nv_bfloat16* k_new; const __nv_bfloat16* v_new;
  const int* slot_ids;
  char* kc; char* vc;
  long long seq_b, head_b;                      // cache strides in bytes (K and V alike)
  int Hq, Hkv, Ls, Lr, max_seqs, nsplit;
  int g;                                        // real group size (<= the kernel's G, which is even)
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
    bulk_g2s(stage + WT_B, vc + (long long)va * ROW_B, bytes, bar);
  }
  const int s2 = max(va, n_low);
  if (s2 < vb) {
    const unsigned bytes = (unsigned)(vb - s2) * ROW_B, off = (unsigned)(s2 - va) * ROW_B;
    const long long src = (long long)(Lsr + s2 - n_low) * ROW_B;
    bulk_g2s(stage + off, kc + src, bytes, bar);
    bulk_g2s(stage + WT_B + off, vc + src, bytes, bar);
  }
}

// packed pairs of floats in one 64-bit register
__device__ __forceinline__ u64 pack2(float lo, float hi) {
  u64 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(u64 v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ u64 fma2(u64 a, u64 b, u64 c) {
  u64 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ u64 mul2(u64 a, u64 b) {
  u64 d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// 8 bf16 (one 128-bit load) -> 4 packed float pairs (elements 2c, 2c+1)
__device__ __forceinline__ void unpack8(const uint4& u, u64 (&f)[4]) {
  f[0] = pack2(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u));
  f[1] = pack2(__uint_as_float(u.y << 16), __uint_as_float(u.y & 0xffff0000u));
  f[2] = pack2(__uint_as_float(u.z << 16), __uint_as_float(u.z & 0xffff0000u));
  f[3] = pack2(__uint_as_float(u.w << 16), __uint_as_float(u.w & 0xffff0000u));
}

template <int G>
__global__ void __launch_bounds__(NT, (G > 4 ? 2 : 3)) decode_gqa_kernel(const FastArgs a) {
  constexpr int VPL = G / 2;                    // logits a lane holds after the reduction
  extern __shared__ __align__(128) unsigned char smem_raw[];
  // [NWARP][NSTAGE] stages | [NWARP][2][8][G][2] probabilities | [NWARP][NSTAGE] mbarriers
  float* pbuf = reinterpret_cast<float*>(smem_raw + NWARP * NSTAGE * STAGE_B);
  uint64_t* bars = reinterpret_cast<uint64_t*>(pbuf + NWARP * 2 * 8 * G * 2);

  const int sp = blockIdx.x, kvh = blockIdx.y, i = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5, hw = lane >> 4, l16 = lane & 15;
  const int odd = l16 & 1, jrow = l16 >> 1;
  asm volatile("griddepcontrol.wait;" ::: "memory");
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
  // even split of this (sequence, KV head)'s 16-row tiles over the splits
  const int ntiles = (n_valid + WT - 1) / WT;
  const int t_begin = (int)((long long)ntiles * sp / a.nsplit);
  const int t_end = (int)((long long)ntiles * (sp + 1) / a.nsplit);
  const int v1 = min(n_valid, t_end * WT);
  // this warp's tiles: t_begin + w, t_begin + w + NWARP, ...
  const int T = t_end - t_begin > w ? (t_end - t_begin - w + NWARP - 1) / NWARP : 0;

  char* kc = a.kc + slot * a.seq_b + kvh * a.head_b;
  char* vc = a.vc + slot * a.seq_b + kvh * a.head_b;
  const __nv_bfloat16* kn = a.k_new ? a.k_new + ((long long)i * a.Hkv + kvh) * D : nullptr;
  const __nv_bfloat16* vn = a.v_new ? a.v_new + ((long long)i * a.Hkv + kvh) * D : nullptr;

  unsigned char* wstages = smem_raw + w * NSTAGE * STAGE_B;
  const uint32_t stage0 = smem_u32(wstages), bar0 = smem_u32(bars + w * NSTAGE);
  if (lane == 0) {
    for (int s = 0; s < NSTAGE; ++s) mbar_init(bar0 + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  if (lane == 0) {
    for (int s = 0; s < NSTAGE && s < T; ++s) {
      const int va = (t_begin + w + s * NWARP) * WT;
      issue_tile(stage0 + s * STAGE_B, bar0 + 8 * s, kc, vc, va, min(v1, va + WT), n_low, Lsr);
    }
  }
  // the CTA that owns the new token's slot stores it (the staged copy is patched below)
  if (new_slot >= t_begin * WT && new_slot < v1 && w == 0) {
    const uint4* srcp = reinterpret_cast<const uint4*>(hw == 0 ? kn : vn);
    char* dst = (hw == 0 ? kc : vc) + (long long)new_slot * ROW_B;
    reinterpret_cast<uint4*>(dst)[l16] = srcp[l16];
  }

  // query rows of the group, pre-scaled so that exp2 can be used directly
  u64 q2[G][4];
  {
    const __nv_bfloat16* qp = a.q + ((long long)i * a.Hq + (long long)kvh * a.g) * D + l16 * 8;
    const u64 sc2 = pack2(a.scale_log2, a.scale_log2);
#pragma unroll
    for (int h = 0; h < G; ++h) {
      // groups of odd size run with one all-zero query row; its result is never written
      const uint4 u = h < a.g ? *reinterpret_cast<const uint4*>(qp + h * D) : make_uint4(0, 0, 0, 0);
      unpack8(u, q2[h]);
#pragma unroll
      for (int c = 0; c < 4; ++c) q2[h][c] = mul2(q2[h][c], sc2);
    }
  }
  u64 acc2[G][4];
  float m_run[G], l_lane[VPL];
#pragma unroll
  for (int h = 0; h < G; ++h) {
    m_run[h] = -INFINITY;
#pragma unroll
    for (int c = 0; c < 4; ++c) acc2[h][c] = 0ull;
  }
#pragma unroll
  for (int e = 0; e < VPL; ++e) l_lane[e] = 0.f;
  float* pw = pbuf + (w * 2 + hw) * 8 * G * 2;  // this half-warp's probabilities [8][G][2]
  bool timed_out = false;

  for (int n = 0; n < T; ++n) {
    const int s = n % NSTAGE;
    const unsigned parity = (unsigned)(n / NSTAGE) & 1u;
    const bool landed = mbar_wait(bar0 + 8 * s, parity);
    if (__any_sync(0xffffffffu, !landed)) { timed_out = true; break; }
    const int va = (t_begin + w + n * NWARP) * WT;
    const int nrows = min(WT, v1 - va);
    unsigned char* sK = wstages + s * STAGE_B;
    unsigned char* sV = sK + WT_B;
    const bool patch = new_slot >= va && new_slot < va + nrows;
    if (patch || nrows < WT) {                   // rare: new-token row, or the ragged last tile
      if (patch)
        reinterpret_cast<uint4*>((hw == 0 ? sK : sV) + (new_slot - va) * ROW_B)[l16] =
            reinterpret_cast<const uint4*>(hw == 0 ? kn : vn)[l16];
      for (int e = lane; e < (WT - nrows) * (ROW_B / 16); e += 32) {      // zero rows past the end
        reinterpret_cast<uint4*>(sK + nrows * ROW_B)[e] = make_uint4(0, 0, 0, 0);
        reinterpret_cast<uint4*>(sV + nrows * ROW_B)[e] = make_uint4(0, 0, 0, 0);
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
    }

    // ---- logits: lane-partial dot products of 8 rows x G heads ----
    float part[8 * G];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const uint4 u = *reinterpret_cast<const uint4*>(sK + (2 * j + hw) * ROW_B + l16 * 16);
      u64 k2[4];
      unpack8(u, k2);
#pragma unroll
      for (int h = 0; h < G; ++h) {
        u64 s2 = mul2(q2[h][0], k2[0]);
#pragma unroll
        for (int c = 1; c < 4; ++c) s2 = fma2(q2[h][c], k2[c], s2);
        float lo, hi;
        unpack2(s2, lo, hi);
        part[j * G + h] = lo + hi;
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
    // lane now holds row 2*jrow + hw of the tile, heads odd*VPL .. odd*VPL + VPL-1
    const bool row_ok = 2 * jrow + hw < nrows;
    // The running maxima are only a reference point for exp2, so they are refreshed lazily:
    // a warp vote detects a logit more than 8 (a factor 256) above the reference, and only then
    // is the max reduced across the warp and the accumulators rescaled.
    bool need = false;
#pragma unroll
    for (int e = 0; e < VPL; ++e) {
      part[e] = row_ok ? part[e] : -INFINITY;
      need |= part[e] > (odd ? m_run[VPL + e] : m_run[e]) + 8.f;
    }
    if (__any_sync(0xffffffffu, need)) {
      float mx[VPL], m_use[G];
#pragma unroll
      for (int e = 0; e < VPL; ++e) {
        mx[e] = part[e];
#pragma unroll
        for (int o = 2; o <= 16; o <<= 1) mx[e] = fmaxf(mx[e], __shfl_xor_sync(0xffffffffu, mx[e], o));
      }
#pragma unroll
      for (int e = 0; e < VPL; ++e) {
        const float other = __shfl_xor_sync(0xffffffffu, mx[e], 1);
        m_use[e] = fmaxf(m_run[e], odd ? other : mx[e]);
        m_use[VPL + e] = fmaxf(m_run[VPL + e], odd ? mx[e] : other);
      }
      float al[G];
#pragma unroll
      for (int h = 0; h < G; ++h) {
        al[h] = m_run[h] == -INFINITY ? 0.f : exp2f(m_run[h] - m_use[h]);
        m_run[h] = m_use[h];
        const u64 al2 = pack2(al[h], al[h]);
#pragma unroll
        for (int c = 0; c < 4; ++c) acc2[h][c] = mul2(acc2[h][c], al2);
      }
#pragma unroll
      for (int e = 0; e < VPL; ++e) l_lane[e] *= odd ? al[VPL + e] : al[e];
    }
#pragma unroll
    for (int e = 0; e < VPL; ++e) {
      const float mh = odd ? m_run[VPL + e] : m_run[e];
      const float p = exp2f(part[e] - (mh == -INFINITY ? 0.f : mh));
      l_lane[e] += p;
      *reinterpret_cast<float2*>(pw + (jrow * G + odd * VPL + e) * 2) = make_float2(p, p);
    }
    __syncwarp();
    // ---- P.V: a lane owns 8 output dims of all G heads ----
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const uint4 u = *reinterpret_cast<const uint4*>(sV + (2 * j + hw) * ROW_B + l16 * 16);
      u64 v2[4];
      unpack8(u, v2);
      const ulonglong2* pp = reinterpret_cast<const ulonglong2*>(pw + j * G * 2);
#pragma unroll
      for (int hp = 0; hp < G / 2; ++hp) {
        const ulonglong2 p2 = pp[hp];             // (p,p) of heads 2hp and 2hp+1
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          acc2[2 * hp][c] = fma2(p2.x, v2[c], acc2[2 * hp][c]);
          acc2[2 * hp + 1][c] = fma2(p2.y, v2[c], acc2[2 * hp + 1][c]);
        }
      }
    }
    __syncwarp();
    if (lane == 0 && n + NSTAGE < T) {
      const int nv = (t_begin + w + (n + NSTAGE) * NWARP) * WT;
      // generic-proxy reads and patches of this stage come before the bulk copy (async proxy) that refills it
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      issue_tile(stage0 + s * STAGE_B, bar0 + 8 * s, kc, vc, nv, min(v1, nv + WT), n_low, Lsr);
    }
  }
  if (timed_out) {
    if (a.status) atomicOr(a.status, SNAP_DEV_WAIT_TIMEOUT);
    // give copies still in flight a bounded chance to land before the stage memory is reused
    for (int s = 0; s < NSTAGE; ++s) (void)mbar_wait(bar0 + 8 * s, 0u);
  }

  // ---- merge the two half-warps, then the warps, and write the split's partial ----
  float acc[G][8];
#pragma unroll
  for (int h = 0; h < G; ++h)
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      unpack2(acc2[h][c], acc[h][2 * c], acc[h][2 * c + 1]);
      acc[h][2 * c] += __shfl_xor_sync(0xffffffffu, acc[h][2 * c], 16);
      acc[h][2 * c + 1] += __shfl_xor_sync(0xffffffffu, acc[h][2 * c + 1], 16);
    }
#pragma unroll
  for (int e = 0; e < VPL; ++e)
#pragma unroll
    for (int o = 2; o <= 16; o <<= 1) l_lane[e] += __shfl_xor_sync(0xffffffffu, l_lane[e], o);
  // every copy this warp issued has been consumed, so its own stage memory is free
  float* wm = reinterpret_cast<float*>(wstages);           // [G] max, [G] sum, [G][D] acc
  float* wl = wm + G;
  float* wacc = wl + G;
  __syncwarp();
  if (lane < 2) {
#pragma unroll
    for (int e = 0; e < VPL; ++e) {
      wm[lane * VPL + e] = lane ? m_run[VPL + e] : m_run[e];
      wl[lane * VPL + e] = l_lane[e];
    }
  }
  if (hw == 0) {
#pragma unroll
    for (int h = 0; h < G; ++h)
#pragma unroll
      for (int c = 0; c < 8; ++c) wacc[h * D + l16 * 8 + c] = acc[h][c];
  }
  __syncthreads();
  float* part_out = a.partials + (((long long)i * a.Hq + (long long)kvh * a.g) * a.nsplit + sp) * PS;
  constexpr int WSTRIDE = NSTAGE * STAGE_B / 4;            // floats between two warps' regions
  const float* base = reinterpret_cast<const float*>(smem_raw);
#pragma unroll
  for (int h = 0; h < G; ++h) {
    float M = -INFINITY;
#pragma unroll
    for (int ww = 0; ww < NWARP; ++ww) M = fmaxf(M, base[ww * WSTRIDE + h]);
    float L = 0.f, O = 0.f;
#pragma unroll
    for (int ww = 0; ww < NWARP; ++ww) {
      const float mw = base[ww * WSTRIDE + h];
      const float f = mw == -INFINITY ? 0.f : exp2f(mw - M);
      L += base[ww * WSTRIDE + G + h] * f;
      O += base[ww * WSTRIDE + 2 * G + h * D + tid] * f;
    }
    if (h < a.g) {
      float* ph = part_out + (long long)h * a.nsplit * PS;
      if (tid == 0) { ph[0] = M; ph[1] = L; }
      ph[2 + tid] = O;
    }
  }
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Merge the splits of one (sequence, query token, query head); maxima are in the log2 domain.
// With q_len query tokens per sequence the rows of `partials` are indexed by sequence * q_len +
// token; the token is token u0 + (its index) of the q_total per sequence in `out`; every token's
// block advances the sequence length by one.
__global__ void __launch_bounds__(D) decode_gqa_merge_kernel(const float* __restrict__ partials,
                                                             __nv_bfloat16* __restrict__ out, int Hq,
                                                             int nsplit, const int* __restrict__ slot_ids,
                                                             int* seq_len, int max_seqs, int bump, int q_len, int q_total,
                                                             int u0) {
  const int h = blockIdx.x, i = blockIdx.y, t = threadIdx.x;
  const long long orow = (long long)(i / q_len) * q_total + u0 + i % q_len;   // token's row of `out`
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const float* p = partials + ((long long)i * Hq + h) * nsplit * PS;
  // launched with programmatic stream serialisation: the grid may start while the split kernel
  // drains; everything the split kernel wrote is visible after this wait
  asm volatile("griddepcontrol.wait;" ::: "memory");
  float M = -INFINITY, L = 0.f, O = 0.f;
  if (nsplit <= D) {
    // The splits' (m, l) are fetched by one thread each; every thread then derives the weights from shared
    // memory and sums its output dim with eight loads in flight (split after split, each thread paid two
    // dependent rounds of global loads per split).
    __shared__ float m_s[D], l_s[D], f_s[D];
    if (t < nsplit) { m_s[t] = p[t * PS]; l_s[t] = p[t * PS + 1]; }
    __syncthreads();
    for (int s = 0; s < nsplit; ++s) M = fmaxf(M, m_s[s]);
    if (t < nsplit) f_s[t] = m_s[t] == -INFINITY ? 0.f : exp2f(m_s[t] - M);
    __syncthreads();
    for (int s = 0; s < nsplit; ++s) L += l_s[s] * f_s[s];
#pragma unroll 8
    for (int s = 0; s < nsplit; ++s) O = fmaf(p[s * PS + 2 + t], f_s[s], O);
  } else {
    for (int s = 0; s < nsplit; ++s) M = fmaxf(M, p[s * PS]);
    for (int s = 0; s < nsplit; ++s) {
      const float ms = p[s * PS];
      const float f = ms == -INFINITY ? 0.f : exp2f(ms - M);
      L += p[s * PS + 1] * f;
      O += p[s * PS + 2 + t] * f;
    }
  }
  out[(orow * Hq + h) * D + t] = __float2bfloat16_rn(L > 0.f ? O / L : 0.f);
  if (bump && h == 0 && t == 0) {
    const int slot = slot_ids[i / q_len];
    if (slot >= 0 && slot < max_seqs) atomicAdd(&seq_len[slot], 1);
  }
}

template <int G>
cudaError_t launch_g(const FastArgs& a, int n_active, __nv_bfloat16* out, int* seq_len, int bump,
                     cudaStream_t st) {
  const size_t smem = (size_t)NWARP * NSTAGE * STAGE_B + NWARP * 2 * 8 * G * 2 * sizeof(float) +
                      NWARP * NSTAGE * 8;
  static SmemLimit limit = {};
  if (cudaError_t e0 = ensure_dyn_smem(decode_gqa_kernel<G>, smem, limit)) return e0;
  // Both kernels are programmatic dependent launches: each may become resident while its
  // predecessor in the stream drains, and waits (griddepcontrol.wait) before touching memory.
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(a.nsplit, a.Hkv, n_active);
  lc.blockDim = dim3(NT);
  lc.dynamicSmemBytes = smem;
  lc.stream = st;
  lc.attrs = attr;
  lc.numAttrs = 1;
  cudaError_t e0 = cudaLaunchKernelEx(&lc, decode_gqa_kernel<G>, a);
  count_launch();
  if (e0 != cudaSuccess) return e0;
  lc.gridDim = dim3(a.Hq, n_active);
  lc.blockDim = dim3(D);
  lc.dynamicSmemBytes = 0;
  const float* parts = a.partials;
  const int* slots = a.slot_ids;
  cudaError_t e = cudaLaunchKernelEx(&lc, decode_gqa_merge_kernel, parts, out, a.Hq, a.nsplit, slots, seq_len,
                                     a.max_seqs, bump, 1, 1, 0);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

// The split merge as a programmatic dependent launch (shared with the tensor-core kernel);
// n_rows = sequences * q_len.
cudaError_t launch_decode_gqa_merge(const float* partials, void* out, int Hq, int nsplit, const int* slot_ids,
                                    int n_rows, int q_len, int* seq_len, int max_seqs, int bump, cudaStream_t st,
                                    int q_total, int u0) {
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(Hq, n_rows);
  lc.blockDim = dim3(D);
  lc.stream = st;
  lc.attrs = attr;
  lc.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&lc, decode_gqa_merge_kernel, partials, static_cast<__nv_bfloat16*>(out), Hq, nsplit,
                                     slot_ids, seq_len, max_seqs, bump, q_len, q_total < q_len ? q_len : q_total,
                                     q_total < q_len ? 0 : u0);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

bool decode_gqa_supported(int dtype, const Shape& s) {
  return dtype == SNAP_BF16 && s.d_qk == D && s.d_v == D && !s.v_aliases_k && s.g >= 1 && s.g <= 8;
}

// Splits per (sequence, KV head).  Measured on B200 over batch sizes 1..64 (5124 slots, 8 KV heads,
// CUDA-graph replays): the time is flat around a total of about 1.75 CTAs per SM for small
// batches -- more splits only lengthen the merge -- and three splits are best once the batch
// alone fills the GPU (they even out the tail).  A split keeps at least two 64-row blocks and,
// for very long caches, at most about 48.
// Option SNAP_OPT_DECODE_NSPLIT overrides the choice (tuning aid).
int decode_gqa_nsplit_for(const Shape& s, int n_active, int sm_count, int ctas_per_sm) {
  const int tiles = (s.Sc + 63) / 64;
  if (const int v = option(SNAP_OPT_DECODE_NSPLIT)) return v < tiles ? v : tiles;
  const long long base = (long long)(n_active > 0 ? n_active : 1) * s.Hkv;
  long long ns = (7LL * sm_count / 4 + base / 2) / base;
  if (ns < 3) ns = 3;
  if (ns <= 6) {
    // Mid-size batches run in one to three waves of CTAs, where a split count that lands just
    // past a wave boundary wastes most of the last wave (20 sequences x 8 KV heads x 3 splits =
    // 480 CTAs on 444 resident slots: 77 us against 69.5 us with 5 splits).  Of 3..6 splits take the
    // one with the fewest wave-rows (waves x rows per split), a little in favour of fewer splits;
    // this reproduces the measured optimum for 8..64 sequences to within 1.5 %.
    const long long slots = (long long)(ctas_per_sm > 0 ? ctas_per_sm : 3) * sm_count;
    const long long penalty = tiles / 20 > 1 ? tiles / 20 : 1;   // a split costs about 1/20 of a pass in set-up and merge
    long long best = 3, best_cost = -1;
    // beyond three waves the hardware's dynamic CTA scheduling evens the tail out and three splits win
    for (long long c = 3; c <= (base * 3 <= 3 * slots ? 6 : 3); ++c) {
      const long long waves = (base * c + slots - 1) / slots;
      const long long cost = waves * ((tiles + c - 1) / c) + c * penalty;
      if (best_cost < 0 || cost < best_cost) { best = c; best_cost = cost; }
    }
    ns = best;
  }
  if (ns < (tiles + 47) / 48) ns = (tiles + 47) / 48;           // very long caches: keep a split short, lengths may be ragged
  if (ns > 16) ns = 16;
  if (ns > tiles / 2) ns = tiles / 2;
  if (ns < 1) ns = 1;
  return (int)ns;
}
int decode_gqa_nsplit(const Shape& s, int n_active, int sm_count) {
  return decode_gqa_nsplit_for(s, n_active, sm_count, s.g > 4 ? 2 : 3);
}
int decode_gqa_mma_nsplit(const Shape& s, int n_active, int sm_count) {
  return decode_gqa_nsplit_for(s, n_active, sm_count, 3);
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
  a.Hq = s.Hq; a.Hkv = s.Hkv; a.Ls = s.Ls; a.Lr = s.Lr; a.max_seqs = s.max_seqs; a.nsplit = nsplit; a.g = s.g;
  a.scale_log2 = s.scale * 1.4426950408889634f;
  a.seq_len = seq_len; a.valid_topk = valid_topk; a.partials = partials; a.status = status;
  __nv_bfloat16* o = static_cast<__nv_bfloat16*>(out);
  const int bump = k_new != nullptr;
  switch (s.g) {
    // the kernel handles an even number of heads per KV head; odd group sizes run padded by one
    case 1: case 2: return launch_g<2>(a, n_active, o, seq_len, bump, st);
    case 3: case 4: return launch_g<4>(a, n_active, o, seq_len, bump, st);
    case 5: case 6: return launch_g<6>(a, n_active, o, seq_len, bump, st);
    case 7: case 8: return launch_g<8>(a, n_active, o, seq_len, bump, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace snap
