// Decode attention over the compressed cache (Section 3.3) for the latent-attention layout on
// tcgen05: one 576-wide cache row shared by all heads, V = its first 512 dims.
//
// With 128 heads sharing every cache row the step is a pair of dense contractions per tile
// (S = Q K^T over 576 dims, O += P V over the tile's rows), so it belongs on the tensor cores.
// Two facts shape the kernel.  The stationary operand, the 128 x 576 query block, would fill
// most of shared memory, so it lives in tensor memory and is the TMEM-sourced A operand of the
// MMAs, as are the probabilities.  And an MMA instruction occupies the tensor pipe for a fixed
// minimum time however few columns it produces (measured: about 110 clocks at N = 32 or 64, from
// either operand source), so tiles are as wide as tensor memory allows:
//     O 128 | S 64 | P 32 (bf16 pairs) | Q 288 (bf16 pairs)    = 512 columns.
// That leaves room for 128 output dims, so the 512 value dims are split over four CTAs that each
// recompute S, and S and P are single-buffered.  Grid = (row splits, 4 x head blocks,
// sequences), one CTA per SM:
//   warp 0      TMA producer: 64-row cache tiles (nine 64-dim slabs, 128-byte swizzle) into a
//               3-stage ring;
//   warp 1      MMA issuer (whole warp converged, instructions predicated on one lane):
//               S(t) = Q K(t)^T is issued as soon as the softmax warps have taken S(t-1) out of
//               tensor memory and runs while they do their arithmetic; O += P(t-1) V(t-1) is
//               queued behind it; V is the same staged tile read as an MN-major operand;
//   warps 2-5   thread = head: read S from TMEM, online softmax in the log2 domain with a lazily
//               refreshed reference (O is rescaled in TMEM only when a logit exceeds it by 8),
//               write P back to TMEM as bf16.
// The new token, if any, is appended by a separate launch before this kernel (Eq. 3).  Every
// mbarrier wait is bounded; one that runs out raises SNAP_DEV_WAIT_TIMEOUT.
#include "snap_internal.cuh"
#include "umma_helpers.cuh"

namespace snap {
namespace {

using namespace umma;

constexpr int DQK = 576, DV = 512, HBLK = 128, TR = 64, NSTG = 3, NTH = 192, DVQ = 128, NQ = DV / DVQ;
constexpr int NSLAB = DQK / 64, SLAB_B = TR * 128, STAGE_B = NSLAB * SLAB_B;        // 9 x 8192 = 73728
constexpr int PSM = DV + 2;
constexpr uint32_t COL_O = 0, COL_S = 128, COL_P = 192, COL_Q = 224;                // tensor-memory columns: O 128 | S 64 | P 32 | Q 288

struct UArgs {
  const __nv_bfloat16* q;
  const int* slot_ids; const int* seq_len; const int* valid_topk;
  int Hq, Ls, Lr, Sc, max_seqs, nsplit;
  float scale_log2;
  float* partials;                             // [n_active][Hq][nsplit][PSM], maxima in the log2 domain
  uint32_t* status;
};

// instruction descriptor: bf16 x bf16 -> fp32, A K-major (tensor memory), B K-major or MN-major
__host__ __device__ constexpr uint32_t idesc_ts(int M, int N, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}
// MN-major operand, 128-byte swizzle: 64 contiguous elements per row of the contraction dim,
// 8-row groups 1024 bytes apart, the next 64 elements `lbo_bytes` further on.
__device__ __forceinline__ uint64_t smem_desc_mn(uint32_t saddr, uint32_t lbo_bytes) {
  return (uint64_t)((saddr >> 4) & 0x3fffu) | ((uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16) |
         ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts_bf16(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
// The same, executed by a whole (converged) warp with the instruction predicated on one lane, so
// that the operands are computed on the warp-uniform path instead of inside a divergent branch.
__device__ __forceinline__ void mma_ts_bf16_pred(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t acc, uint32_t leader) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %4, 0;\n\tsetp.ne.b32 q, %5, 0;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc), "r"(leader) : "memory");
}
__device__ __forceinline__ void mma_commit_pred(uint32_t bar, uint32_t leader) {
  asm volatile(
      "{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
      "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
      ::"r"(bar), "r"(leader) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// Bounded wait whose outcome is the same for every lane (what follows is warp-collective).
__device__ __forceinline__ bool wait_warp(uint32_t bar, unsigned parity, volatile int* abort_flag) {
  return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
}

// Tile g of a sequence: rows [row0, row0 + TR) of the cache, valid below row_end.  Tiles cover
// [0, n_low) first, then [Lsr, Lsr + n_top).
struct TileRows { int row0, row_end; };
__device__ __forceinline__ TileRows tile_rows(int g, int nA, int n_low, int Lsr, int n_top) {
  TileRows t;
  if (g < nA) { t.row0 = g * TR; t.row_end = n_low; }
  else { t.row0 = Lsr + (g - nA) * TR; t.row_end = Lsr + n_top; }
  return t;
}

__global__ void __launch_bounds__(NTH, 1) decode_mla_umma_kernel(const UArgs a, const __grid_constant__ CUtensorMap tmap_c) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* Ks = smem;                                                   // [NSTG][9 slabs][32 rows][128 B]
  uint64_t* bars = reinterpret_cast<uint64_t*>(Ks + NSTG * STAGE_B);
  // full[NSTG] empty[NSTG] s_full s_free p_ready pv_done q_ready
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * NSTG + 5);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int sp = blockIdx.x, hb = blockIdx.y / NQ, qd = blockIdx.y % NQ, i = blockIdx.z;
  const int slot = a.slot_ids[i];
  const bool bad = slot < 0 || slot >= a.max_seqs;
  const int Lsr = a.Ls + a.Lr;
  int n_low = 0, n_top = 0;
  if (!bad) {
    n_low = min(a.seq_len[slot], Lsr);
    n_top = a.valid_topk[slot];
  } else if (tid == 0 && sp == 0 && blockIdx.y == 0 && a.status) {
    atomicOr(a.status, SNAP_DEV_BAD_SLOT);
  }
  const int nA = (n_low + TR - 1) / TR, ntiles = nA + (n_top + TR - 1) / TR;
  const int g0 = (int)((long long)ntiles * sp / a.nsplit);
  const int g1 = (int)((long long)ntiles * (sp + 1) / a.nsplit);
  const int nt = g1 - g0;

  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8 * s; };
  auto empty_bar = [&](int s) { return bar0 + 8 * (NSTG + s); };
  const uint32_t sfull_bar = bar0 + 8 * (2 * NSTG), sfree_bar = bar0 + 8 * (2 * NSTG + 1);
  const uint32_t pready_bar = bar0 + 8 * (2 * NSTG + 2), pvdone_bar = bar0 + 8 * (2 * NSTG + 3);
  const uint32_t qready_bar = bar0 + 8 * (2 * NSTG + 4);

  if (tid == 0) {
    *abort_flag = 0;
    for (int s = 0; s < NSTG; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(sfull_bar, 1); mbar_init(sfree_bar, 4); mbar_init(pready_bar, 4); mbar_init(pvdone_bar, 1);
    mbar_init(qready_bar, 4);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      bool ok = true;
      for (int it = 0; it < nt && ok; ++it) {
        const int s = it % NSTG;
        if (!mbar_wait(empty_bar(s), ((unsigned)(it / NSTG) & 1u) ^ 1u, abort_flag)) { *abort_flag = 1; ok = false; break; }
        const TileRows tr = tile_rows(g0 + it, nA, n_low, Lsr, n_top);
        mbar_expect_tx(full_bar(s), (unsigned)STAGE_B);
        for (int h = 0; h < NSLAB; ++h)
          tma_load_3d(smem_u32(Ks) + s * STAGE_B + h * SLAB_B, &tmap_c, h * 64, tr.row0, slot, full_bar(s));
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (nt > 0) {                                              // whole warp, MMAs and commits predicated on lane 0
      const uint32_t leader = lane == 0;
      const uint32_t idesc_s = idesc_ts(128, TR, false), idesc_pv = idesc_ts(128, DVQ, true);
      bool ok = wait_warp(qready_bar, 0u, abort_flag);
      fence_after();
      // S, P and the one set of barriers around them are single-buffered: tile it's logits are
      // computed once the softmax warps have taken tile it-1's out of tensor memory, and run on the
      // tensor pipe while those warps do their arithmetic; O += P(it-1) V(it-1) is queued behind.
      auto issue_pv = [&](int it) -> bool {                   // O += P(it) V(it): V = rows of the staged tile, MN-major
        if (!wait_warp(pready_bar, (unsigned)it & 1u, abort_flag)) return false;
        fence_after();
        const int s = it % NSTG;
        const uint32_t vst = smem_u32(Ks) + s * STAGE_B + (2 * qd) * SLAB_B;
#pragma unroll
        for (int ks = 0; ks < TR / 16; ++ks)
          mma_ts_bf16_pred(tmem_base + COL_O, tmem_base + COL_P + 8 * ks, smem_desc_mn(vst + ks * 16 * 128, SLAB_B),
                           idesc_pv, (it | ks) != 0, leader);
        mma_commit_pred(pvdone_bar, leader);
        mma_commit_pred(empty_bar(s), leader);                 // the stage may be refilled once these MMAs have read it
        return true;
      };
      for (int it = 0; it < nt && ok; ++it) {
        const int s = it % NSTG;
        ok = wait_warp(full_bar(s), (unsigned)(it / NSTG) & 1u, abort_flag);
        if (ok && it > 0) ok = wait_warp(sfree_bar, (unsigned)(it - 1) & 1u, abort_flag);
        if (!ok) break;
        fence_after();
        // descriptors differ from the stage's first one only by compile-time constants (16-byte units)
        const uint64_t kd0 = smem_desc(smem_u32(Ks) + s * STAGE_B);
        const uint32_t sd = tmem_base + COL_S, qa = tmem_base + COL_Q;
#pragma unroll
        for (int k = 0; k < NSLAB * 4; ++k)                    // S = Q K(it)^T
          mma_ts_bf16_pred(sd, qa + 8 * k, kd0 + (uint64_t)(((k >> 2) * SLAB_B + (k & 3) * 32) >> 4), idesc_s, k != 0, leader);
        mma_commit_pred(sfull_bar, leader);
        if (it > 0) ok = issue_pv(it - 1);
      }
      if (ok) ok = issue_pv(nt - 1);
      if (!ok && lane == 0) *abort_flag = 1;
    }
  } else {
    // ---------------- softmax warps: thread = head ----------------
    const int hrow = 32 * (warp & 3) + lane;                   // TMEM lane = head within the block
    const uint32_t lane_addr = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16);
    const int head = hb * HBLK + hrow;
    float m_ref = -INFINITY, l_sum = 0.f;
    bool ok = true;
    if (nt > 0) {
      // query row -> tensor memory (two bf16 per 32-bit column, dims in order)
      const uint4* qrow = reinterpret_cast<const uint4*>(a.q + ((long long)i * a.Hq + head) * DQK);
      // six 16-column groups per round so that 24 row loads are in flight at a time
#pragma unroll 1
      for (int c0 = 0; c0 < DQK / 32; c0 += 6) {
        uint4 u[24];
#pragma unroll
        for (int e = 0; e < 24; ++e) u[e] = qrow[4 * c0 + e];
#pragma unroll
        for (int c = 0; c < 6; ++c) {
          uint32_t r[16];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            r[4 * e] = u[4 * c + e].x; r[4 * e + 1] = u[4 * c + e].y; r[4 * e + 2] = u[4 * c + e].z; r[4 * e + 3] = u[4 * c + e].w;
          }
          tmem_st16(lane_addr + COL_Q + 16 * (c0 + c), r);
        }
      }
      tmem_st_wait();
      fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(qready_bar);
    }
    for (int it = 0; it < nt; ++it) {
      if (!wait_warp(sfull_bar, (unsigned)it & 1u, abort_flag)) { ok = false; break; }
      fence_after();
      uint32_t r0[16], r1[16], r2[16], r3[16];
      tmem_ld16_issue(lane_addr + COL_S, r0);
      tmem_ld16_issue(lane_addr + COL_S + 16, r1);
      tmem_ld16_issue(lane_addr + COL_S + 32, r2);
      tmem_ld16_issue(lane_addr + COL_S + 48, r3);
      const TileRows tr = tile_rows(g0 + it, nA, n_low, Lsr, n_top);
      const int nrows = tr.row_end - tr.row0;                  // >= 1; columns at or past it are masked
      tmem_ld16_wait(r0); tmem_ld16_wait(r1); tmem_ld16_wait(r2); tmem_ld16_wait(r3);
      fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(sfree_bar);                   // the next tile's logits may overwrite S
      float v[TR];
      float mx = -INFINITY;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        v[j] = j < nrows ? __uint_as_float(r0[j]) * a.scale_log2 : -INFINITY;
        v[16 + j] = 16 + j < nrows ? __uint_as_float(r1[j]) * a.scale_log2 : -INFINITY;
        v[32 + j] = 32 + j < nrows ? __uint_as_float(r2[j]) * a.scale_log2 : -INFINITY;
        v[48 + j] = 48 + j < nrows ? __uint_as_float(r3[j]) * a.scale_log2 : -INFINITY;
        mx = fmaxf(fmaxf(mx, fmaxf(v[j], v[16 + j])), fmaxf(v[32 + j], v[48 + j]));
      }
      // Lazy reference: refreshed (and O rescaled) only when some head of the warp sees a logit 8
      // above its reference; the tensor-memory accesses are warp-collective, so the warp votes.
      bool pv_waited = it == 0;
      if (__any_sync(0xffffffffu, mx > m_ref + 8.f)) {
        const float m_new = fmaxf(m_ref, mx);
        const float alpha = m_ref == -INFINITY ? 0.f : exp2f(m_ref - m_new);
        if (it > 0) {
          if (!wait_warp(pvdone_bar, (unsigned)(it - 1) & 1u, abort_flag)) { ok = false; break; }
          pv_waited = true;
          fence_after();
#pragma unroll 1
          for (int c = 0; c < DVQ / 16; ++c) {
            uint32_t o[16];
            tmem_ld16_issue(lane_addr + COL_O + 16 * c, o);
            tmem_ld16_wait(o);
#pragma unroll
            for (int e = 0; e < 16; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st16(lane_addr + COL_O + 16 * c, o);
          }
          tmem_st_wait();
        }
        l_sum *= alpha;
        m_ref = m_new;
      }
      uint32_t pk0[16], pk1[16];
      const float mr = m_ref == -INFINITY ? 0.f : m_ref;
      float ls0 = 0.f, ls1 = 0.f;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const float p0 = fast_exp2(v[2 * j] - mr), p1 = fast_exp2(v[2 * j + 1] - mr);
        const float p2 = fast_exp2(v[32 + 2 * j] - mr), p3 = fast_exp2(v[33 + 2 * j] - mr);
        ls0 += p0 + p1;
        ls1 += p2 + p3;
        pk0[j] = pack_bf16(p0, p1);
        pk1[j] = pack_bf16(p2, p3);
      }
      l_sum += ls0 + ls1;
      if (!pv_waited) {                                        // P was last read by the MMAs of tile it - 1
        if (!wait_warp(pvdone_bar, (unsigned)(it - 1) & 1u, abort_flag)) { ok = false; break; }
        fence_after();
      }
      tmem_st16(lane_addr + COL_P, pk0);
      tmem_st16(lane_addr + COL_P + 16, pk1);
      tmem_st_wait();
      fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(pready_bar);
    }
    if (!ok) *abort_flag = 1;
    // ---------------- this split's partial result ----------------
    float* ph = a.partials + (((long long)i * a.Hq + head) * a.nsplit + sp) * PSM;
    if (ok && nt > 0) ok = wait_warp(pvdone_bar, (unsigned)(nt - 1) & 1u, abort_flag);
    if (!ok) *abort_flag = 1;
    fence_after();
    if (qd == 0) { ph[0] = nt > 0 && ok ? m_ref : -INFINITY; ph[1] = nt > 0 && ok ? l_sum : 0.f; }
    // warp-uniform: nt and the outcome of the waits are the same for the whole warp up to the vote
    const bool have = __all_sync(0xffffffffu, ok && nt > 0);
#pragma unroll 1
    for (int c = 0; c < DVQ / 16; ++c) {
      uint32_t o[16];
      if (have) {
        tmem_ld16_issue(lane_addr + COL_O + 16 * c, o);
        tmem_ld16_wait(o);
      } else {
#pragma unroll
        for (int e = 0; e < 16; ++e) o[e] = 0u;
      }
      float2* d2 = reinterpret_cast<float2*>(ph + 2 + qd * DVQ + 16 * c);   // ph + 2 is 8-byte aligned only
#pragma unroll
      for (int e = 0; e < 8; ++e) d2[e] = make_float2(__uint_as_float(o[2 * e]), __uint_as_float(o[2 * e + 1]));
    }
  }

  fence_before();
  __syncthreads();
  fence_after();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  if (tid == 0 && *abort_flag && a.status) atomicOr(a.status, SNAP_DEV_WAIT_TIMEOUT);
}

size_t umma_smem_bytes() { return (size_t)NSTG * STAGE_B + (2 * NSTG + 7) * 8 + 16 + 1024; }

}  // namespace

bool decode_mla_umma_supported(int dtype, const Shape& s) {
  return dtype == SNAP_BF16 && s.v_aliases_k && s.d_qk == DQK && s.d_v == DV && s.Hkv == 1 && s.Hq % HBLK == 0 &&
         umma::encode_tiled_fn() != nullptr;
}

// Row splits per sequence: the grid (splits x 4 value quarters x head blocks x sequences) should
// fill the SMs once or twice over, with at least four tiles per split.
int decode_mla_umma_nsplit(const Shape& s, int n_active, int sm_count) {
  const int tiles = (s.Sc + TR - 1) / TR + 1;
  const long long base = (long long)n_active * NQ * (s.Hq / HBLK);
  int best = 1;
  double best_fill = -1.0;
  for (int ns = 1; ns <= 64 && ns <= (tiles / 4 > 1 ? tiles / 4 : 1); ++ns) {
    const long long ctas = base * ns;
    const long long waves = (ctas + sm_count - 1) / sm_count;
    if (waves > 2 && ns > 1) break;
    const double fill = (double)ctas / (double)(waves * sm_count);
    if (fill > best_fill + 1e-9) { best_fill = fill; best = ns; }
  }
  return best;
}

size_t decode_mla_umma_partial_floats(const Shape& s, int n_active, int nsplit) {
  return (size_t)n_active * s.Hq * nsplit * PSM;
}

cudaError_t launch_decode_mla_umma(const Shape& s, const void* q, const void* k_new, const int* slot_ids,
                                   int n_active, void* k_cache, int* seq_len, const int* valid_topk, void* out,
                                   float* partials, int nsplit, uint32_t* status, cudaStream_t st) {
  if (n_active == 0) return cudaSuccess;
  umma::EncodeTiledFn enc = umma::encode_tiled_fn();
  if (!enc) return cudaErrorNotSupported;
  if (k_new) {                                                 // Eq. 3 append (also advances the lengths)
    cudaError_t e = launch_append(SNAP_BF16, s, k_new, nullptr, slot_ids, n_active, k_cache, nullptr, seq_len, status, st);
    if (e != cudaSuccess) return e;
  }
  CUtensorMap tc;
  const cuuint64_t dims[3] = {(cuuint64_t)DQK, (cuuint64_t)s.Sc, (cuuint64_t)s.max_seqs};
  const cuuint64_t strides[2] = {(cuuint64_t)DQK * 2, (cuuint64_t)s.Sc * DQK * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)TR, 1}, estr[3] = {1, 1, 1};
  if (enc(&tc, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, k_cache, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  UArgs a;
  a.q = static_cast<const __nv_bfloat16*>(q);
  a.slot_ids = slot_ids; a.seq_len = seq_len; a.valid_topk = valid_topk;
  a.Hq = s.Hq; a.Ls = s.Ls; a.Lr = s.Lr; a.Sc = s.Sc; a.max_seqs = s.max_seqs; a.nsplit = nsplit;
  a.scale_log2 = s.scale * 1.4426950408889634f;
  a.partials = partials; a.status = status;
  const size_t smem = umma_smem_bytes();
  static SmemLimit limit = {};
  if (cudaError_t e = ensure_dyn_smem(decode_mla_umma_kernel, smem, limit)) return e;
  dim3 grid(nsplit, NQ * (s.Hq / HBLK), n_active);
  decode_mla_umma_kernel<<<grid, NTH, smem, st>>>(a, tc);
  count_launch();
  return launch_decode_mla_merge(partials, out, n_active, s.Hq, nsplit, slot_ids, seq_len, s.max_seqs, 0, st);
}

}  // namespace snap
