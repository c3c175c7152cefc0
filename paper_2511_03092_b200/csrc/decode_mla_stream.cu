// Decode attention over the compressed cache (Section 3.3) for the latent-attention layout on
// tcgen05, streamed version: one 576-wide cache row shared by all heads, V = its first 512 dims.
//
// An MMA instruction occupies the tensor pipe for a fixed minimum time however few columns it
// produces, so this kernel is built around wide instructions: S = Q K^T in 128-row tiles
// (N = 128) and O += P V over 256 value dims at a time (N = 256).  The 128 x 576 query block
// stays in shared memory (nine 64-dim slabs, 128-byte swizzle) as the A operand of S; what is
// left of shared memory is a ring of five 16 KB stages through which the cache rows stream
// twice: as key slabs (128 rows x 64 dims, K-major B operand of S) and, once the tile's
// probabilities exist, as value chunks (32 rows x 256 dims, MN-major B operand of P V).  The
// second pass costs 0.44 of the first in L2 traffic and buys a tile four times as wide as one
// that has to stay resident.  Tensor memory holds S twice (2 x 128 columns, so that the next
// tile's logits are computed while the softmax warps work on this one) and O (256 columns: the
// 512 value dims are split over two CTAs that each compute S); the probabilities overwrite
// their own logits as bf16 pairs and are the TMEM-sourced A operand of P V.
//
// Grid = (row splits, 2 x head blocks, sequences), one CTA per SM:
//   warp 0      TMA producer, in the order the MMAs consume: K(0), K(1), V(0), K(2), V(1), ...
//   warp 1      MMA issuer (whole warp converged, instructions predicated on one lane)
//   warps 2-5   thread = head: S from TMEM, online softmax in the log2 domain with a lazily
//               refreshed reference (O is rescaled in TMEM only when a logit exceeds it by 8),
//               P back to TMEM.
// The new token, if any, is appended here (Eq. 3): the CTAs whose tile range holds its slot
// patch the row into their staged key slabs and value chunks before the tensor core reads them
// (nobody else loads that row), one of them stores it to the cache, and the merge kernel
// advances the length.  Every mbarrier wait is bounded; one that runs out raises
// SNAP_DEV_WAIT_TIMEOUT.
#include "snap_internal.cuh"
#include "umma_helpers.cuh"

namespace snap {
namespace {

using namespace umma;

constexpr int DQK = 576, DV = 512, HBLK = 128, TR = 128, NSTG = 5, NTH = 192, DVH = 256, NHALF = DV / DVH;
constexpr int NSLAB = DQK / 64, QSLAB_B = HBLK * 128, STAGE_B = 16384;   // key slab = 128 rows x 128 B = one stage
constexpr int VROWS = 32, VSUB_B = VROWS * 128, NVCH = TR / VROWS;       // value chunk = 4 sub-slabs of 32 rows x 64 dims
constexpr int PSM = DV + 4;                                              // m, l, two unused, acc[DV]: rows 16-byte aligned
constexpr uint32_t COL_S = 0, COL_O = 256;                               // tensor memory: S0 128 | S1 128 | O 256

struct SArgs {
  const __nv_bfloat16* k_new;                  // NULL, or [n_active][576]: the new token's row, appended here (Eq. 3)
  unsigned char* kc;                           // the cache, for the one global store of that row
  const int* slot_ids; const int* seq_len; const int* valid_topk;
  int Hq, Ls, Lr, Sc, max_seqs, nsplit;
  long long knew_seq_stride;                   // elements between two sequences' new rows
  float scale_log2;
  float* partials;                             // [n_active][Hq][nsplit][PSM], maxima in the log2 domain
  uint32_t* status;
};

// Tile g of a sequence: rows [row0, row0 + TR) of the cache, valid below row_end.  Tiles cover
// [0, n_low) first, then [Lsr, Lsr + n_top).
struct TileRows { int row0, row_end; };
__device__ __forceinline__ TileRows tile_rows(int g, int nA, int n_low, int Lsr, int n_top) {
  TileRows t;
  if (g < nA) { t.row0 = g * TR; t.row_end = n_low; }
  else { t.row0 = Lsr + (g - nA) * TR; t.row_end = Lsr + n_top; }
  return t;
}

__global__ void __launch_bounds__(NTH, 1)
decode_mla_stream_kernel(const SArgs a, const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                         const __grid_constant__ CUtensorMap tmap_v) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* Qs = smem;                                                   // [9 slabs][128 heads][128 B]
  unsigned char* Rs = Qs + NSLAB * QSLAB_B;                                   // [NSTG][16 KB] ring
  uint64_t* bars = reinterpret_cast<uint64_t*>(Rs + NSTG * STAGE_B);
  // full[NSTG] empty[NSTG] s_full[2] p_ready[2] pv_done[2] q_full
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * NSTG + 7);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int sp = blockIdx.x, hb = blockIdx.y / NHALF, hd = blockIdx.y % NHALF, i = blockIdx.z;
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8 * s; };
  auto empty_bar = [&](int s) { return bar0 + 8 * (NSTG + s); };
  auto sfull_bar = [&](int b) { return bar0 + 8 * (2 * NSTG + b); };
  auto pready_bar = [&](int b) { return bar0 + 8 * (2 * NSTG + 2 + b); };
  auto pvdone_bar = [&](int b) { return bar0 + 8 * (2 * NSTG + 4 + b); };
  const uint32_t qfull_bar = bar0 + 8 * (2 * NSTG + 6);

  if (tid == 0) {
    *abort_flag = 0;
    for (int s = 0; s < NSTG; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(sfull_bar(b), 1); mbar_init(pready_bar(b), 4); mbar_init(pvdone_bar(b), 1); }
    mbar_init(qfull_bar, 1);
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

  // launched as a programmatic dependent of whatever precedes it: the set-up above overlaps that
  // kernel's tail; wait for it before reading lengths or rows
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int slot = a.slot_ids[i];
  const bool bad = slot < 0 || slot >= a.max_seqs;
  const int Lsr = a.Ls + a.Lr;
  int n_low = 0, n_top = 0, new_slot = -1;
  if (!bad) {
    int len = a.seq_len[slot];
    if (a.k_new) { new_slot = ring_slot(len, a.Ls, a.Lr); ++len; }   // the token being written sees itself
    n_low = min(len, Lsr);
    n_top = a.valid_topk[slot];
  } else if (tid == 0 && sp == 0 && blockIdx.y == 0 && a.status) {
    atomicOr(a.status, SNAP_DEV_BAD_SLOT);
  }
  const int nA = (n_low + TR - 1) / TR, ntiles = nA + (n_top + TR - 1) / TR;
  const int g0 = (int)((long long)ntiles * sp / a.nsplit);
  const int g1 = (int)((long long)ntiles * (sp + 1) / a.nsplit);
  const int nt = g1 - g0;
  // the new row lies in the low section (sinks or ring): tile new_slot / TR, if this split has it
  const int it_new = new_slot >= 0 && new_slot / TR >= g0 && new_slot / TR < g1 ? new_slot / TR - g0 : -1;
  const int r_new = new_slot - (g0 + it_new) * TR;             // its row within that tile
  const uint4* knew4 = a.k_new ? reinterpret_cast<const uint4*>(a.k_new + (long long)i * a.knew_seq_stride) : nullptr;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0 && nt > 0) {
      mbar_expect_tx(qfull_bar, (unsigned)NSLAB * QSLAB_B);
      for (int h = 0; h < NSLAB; ++h)
        tma_load_3d(smem_u32(Qs) + h * QSLAB_B, &tmap_q, h * 64, hb * HBLK, i, qfull_bar);
      int s = 0;                                               // stage filled next
      unsigned ph = 1u;                                        // parity of its "free" phase
      uint32_t fb = full_bar(0), dst = smem_u32(Rs);
      bool ok = true;
      auto stage_wait = [&]() -> bool {
        if (!mbar_wait(fb + 8 * NSTG, ph, abort_flag)) { *abort_flag = 1; return false; }
        mbar_expect_tx(fb, (unsigned)STAGE_B);
        return true;
      };
      auto advance = [&]() {
        if (++s == NSTG) { s = 0; ph ^= 1u; fb = full_bar(0); dst = smem_u32(Rs); }
        else { fb += 8; dst += STAGE_B; }
      };
      auto load_k = [&](int it) {                              // nine key slabs of tile it
        const TileRows tr = tile_rows(g0 + it, nA, n_low, Lsr, n_top);
        for (int h = 0; h < NSLAB && ok; ++h) {
          ok = stage_wait();
          if (!ok) break;
          tma_load_3d(dst, &tmap_k, h * 64, tr.row0, slot, fb);
          advance();
        }
      };
      auto load_v = [&](int it) {                              // four value chunks of tile it (this CTA's 256 dims)
        const TileRows tr = tile_rows(g0 + it, nA, n_low, Lsr, n_top);
        for (int c = 0; c < NVCH && ok; ++c) {
          ok = stage_wait();
          if (!ok) break;
          for (int j = 0; j < DVH / 64; ++j)
            tma_load_3d(dst + j * VSUB_B, &tmap_v, hd * DVH + j * 64, tr.row0 + c * VROWS, slot, fb);
          advance();
        }
      };
      load_k(0);
      for (int it = 0; it < nt && ok; ++it) {
        if (it + 1 < nt) load_k(it + 1);
        if (ok) load_v(it);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (nt > 0) {
      const uint32_t leader = lane == 0;
      const uint32_t idesc_s = idesc_f16(128, TR, false), idesc_pv = idesc_f16(128, DVH, true);
      const uint64_t qd0 = smem_desc(smem_u32(Qs)), kd0 = smem_desc(smem_u32(Rs)), vd0 = smem_desc_mn(smem_u32(Rs), VSUB_B);
      // The stage index, its phase and its barrier are carried along and the descriptors advance by
      // additions: this warp's instruction chain per stage is what the tensor pipe waits for.
      int s = 0;                                               // stage consumed next
      unsigned ph = 0u;                                        // parity of its "landed" phase
      uint32_t fb = full_bar(0);
      auto advance = [&]() {
        if (++s == NSTG) { s = 0; ph ^= 1u; fb = full_bar(0); }
        else fb += 8;
      };
      bool ok = wait_warp(qfull_bar, 0u, abort_flag);
      fence_after();
      auto issue_s = [&](int it) -> bool {                    // S[it & 1] = Q K(it)^T, one key slab per stage
        const uint32_t sd = tmem_base + COL_S + (it & 1) * TR;
        uint64_t qd = qd0;
#pragma unroll 1
        for (int h = 0; h < NSLAB; ++h, qd += QSLAB_B >> 4) {
          if (!wait_warp(fb, ph, abort_flag)) return false;
          if (it == it_new) {
            // the new token's row: eight 16-byte chunks of this 64-dim slab, at their swizzled places
            if (lane < 8)
              *reinterpret_cast<uint4*>(Rs + s * STAGE_B + r_new * 128 + ((lane ^ (r_new & 7)) << 4)) = knew4[h * 8 + lane];
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
          }
          mma_ss_slab4_pred(sd, qd, kd0 + (uint64_t)(s * (STAGE_B >> 4)), idesc_s, h != 0, leader);
          commit_pred(fb + 8 * NSTG, leader);
          advance();
        }
        commit_pred(sfull_bar(it & 1), leader);
        return true;
      };
      if (ok) ok = issue_s(0);
      for (int it = 0; it < nt && ok; ++it) {
        const int b = it & 1;
        if (it + 1 < nt) { ok = issue_s(it + 1); if (!ok) break; }
        ok = wait_warp(pready_bar(b), (unsigned)(it / 2) & 1u, abort_flag);
        if (!ok) break;
        fence_after();
        const uint32_t pa = tmem_base + COL_S + b * TR;       // P(it) lies over the first 64 columns of S(it)
        const TileRows ptr_ = tile_rows(g0 + it, nA, n_low, Lsr, n_top);
        const int tile_nrows = ptr_.row_end - ptr_.row0;
#pragma unroll 1
        for (int c = 0; c < NVCH; ++c) {                      // O += P(it) V(it), one 32-row value chunk per stage
          ok = wait_warp(fb, ph, abort_flag);
          if (!ok) break;
          if (tile_nrows < (c + 1) * VROWS) {
            // ragged chunk: rows past the end may hold anything (memory the caller never wrote), and a
            // zero probability does not silence a NaN in V: clear them before the tensor core reads
            const int first = max(tile_nrows - c * VROWS, 0);
            for (int e = lane; e < (VROWS - first) * (DVH / 64) * 8; e += 32) {
              const int r = first + e / ((DVH / 64) * 8), j = (e / 8) % (DVH / 64), ch = e % 8;
              *reinterpret_cast<uint4*>(Rs + s * STAGE_B + j * VSUB_B + r * 128 + ch * 16) = make_uint4(0, 0, 0, 0);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
          }
          if (it == it_new && r_new / VROWS == c) {
            // the new row as a value row: this CTA's 256 dims = 4 sub-slabs x 8 chunks, one per lane
            const int rr = r_new % VROWS, j = lane >> 3, ch = lane & 7;
            *reinterpret_cast<uint4*>(Rs + s * STAGE_B + j * VSUB_B + rr * 128 + ((ch ^ (rr & 7)) << 4)) =
                knew4[(hd * DVH + j * 64) / 8 + ch];
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
          }
          static_assert(VROWS == 32, "two 16-row steps per value chunk");
          mma_ts_2_pred(tmem_base + COL_O, pa + 16 * c, vd0 + (uint64_t)(s * (STAGE_B >> 4)), (16 * 128) >> 4, idesc_pv, (it | c) != 0,
                        leader);
          commit_pred(fb + 8 * NSTG, leader);
          advance();
        }
        if (ok) commit_pred(pvdone_bar(b), leader);
      }
      if (!ok && lane == 0) *abort_flag = 1;
    }
  } else {
    // ---------------- softmax warps: thread = head ----------------
    const int hrow = 32 * (warp & 3) + lane;                   // TMEM lane = head within the block
    if (it_new >= 0 && hd == 0 && hb == 0 && hrow < DQK / 8)   // the one store of the new row to the cache
      reinterpret_cast<uint4*>(a.kc + ((long long)slot * a.Sc + new_slot) * (DQK * 2))[hrow] = knew4[hrow];
    const uint32_t lane_addr = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16);
    const int head = hb * HBLK + hrow;
    float m_ref = -INFINITY, l_sum = 0.f;
    bool ok = true;
    for (int it = 0; it < nt; ++it) {
      const int b = it & 1;
      if (!wait_warp(sfull_bar(b), (unsigned)(it / 2) & 1u, abort_flag)) { ok = false; break; }
      fence_after();
      const uint32_t s_addr = lane_addr + COL_S + b * TR;
      const TileRows tr = tile_rows(g0 + it, nA, n_low, Lsr, n_top);
      const int nrows = tr.row_end - tr.row0;                  // >= 1; columns at or past it are masked
      float v[TR];                                             // raw logits
      {
        // all eight loads in flight before the one wait: the tensor-memory latency is paid once per tile
        uint32_t r[8][16];
#pragma unroll
        for (int c = 0; c < 8; ++c) tmem_ld16_issue(s_addr + 16 * c, r[c]);
#pragma unroll
        for (int c = 0; c < 8; ++c) tmem_ld16_wait(r[c]);
#pragma unroll
        for (int c = 0; c < 8; ++c)
#pragma unroll
          for (int j = 0; j < 16; ++j) v[16 * c + j] = __uint_as_float(r[c][j]);
      }
      if (nrows < TR) {                                        // ragged tile: columns at or past nrows are masked
#pragma unroll
        for (int j = 0; j < TR; ++j) v[j] = j < nrows ? v[j] : -INFINITY;
      }
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int j = 0; j < TR; j += 4) {
        mx0 = fmaxf(mx0, fmaxf(v[j], v[j + 1]));
        mx1 = fmaxf(mx1, fmaxf(v[j + 2], v[j + 3]));
      }
      const float mx = fmaxf(mx0, mx1) * a.scale_log2;         // scale > 0: the largest raw logit is the largest scaled one
      // Lazy reference: refreshed (and O rescaled) only when some head of the warp sees a logit 8
      // above its reference; the tensor-memory accesses are warp-collective, so the warp votes.
      if (__any_sync(0xffffffffu, mx > m_ref + 8.f)) {
        const float m_new = fmaxf(m_ref, mx);
        const float alpha = m_ref == -INFINITY ? 0.f : exp2f(m_ref - m_new);
        if (it > 0) {
          if (!wait_warp(pvdone_bar((it - 1) & 1), (unsigned)((it - 1) / 2) & 1u, abort_flag)) { ok = false; break; }
          fence_after();
#pragma unroll 1
          for (int c = 0; c < DVH / 16; ++c) {
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
      const float nmr = m_ref == -INFINITY ? 0.f : -m_ref;
      // the logits of this tile are all in registers, so the probabilities may overwrite them;
      // two-wide packed multiply-adds and sums around the exponentials
      const u64 sc2 = pack2(a.scale_log2, a.scale_log2), nmr2 = pack2(nmr, nmr);
      u64 ls2 = pack2(0.f, 0.f);
#pragma unroll
      for (int c = 0; c < TR / 32; ++c) {
        uint32_t pk[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const u64 x2 = fma2(pack2(v[32 * c + 2 * j], v[32 * c + 2 * j + 1]), sc2, nmr2);
          const float p0 = fast_exp2(lo2(x2)), p1 = fast_exp2(hi2(x2));
          ls2 = add2(ls2, pack2(p0, p1));
          pk[j] = pack_bf16(p0, p1);
        }
        tmem_st16(s_addr + 16 * c, pk);
      }
      l_sum += lo2(ls2) + hi2(ls2);
      tmem_st_wait();
      fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(pready_bar(b));
    }
    if (!ok) *abort_flag = 1;
    // ---------------- this split's partial result ----------------
    float* ph = a.partials + (((long long)i * a.Hq + head) * a.nsplit + sp) * PSM;
    if (ok && nt > 0) ok = wait_warp(pvdone_bar((nt - 1) & 1), (unsigned)((nt - 1) / 2) & 1u, abort_flag);
    if (!ok) *abort_flag = 1;
    fence_after();
    if (hd == 0) { ph[0] = nt > 0 && ok ? m_ref : -INFINITY; ph[1] = nt > 0 && ok ? l_sum : 0.f; }
    const bool have = __all_sync(0xffffffffu, ok && nt > 0);
    // O goes out 32 columns at a time through this warp's corner of the (now idle) ring, transposed so that
    // a store instruction writes four heads' 128-byte runs instead of 32 scattered pieces
    float* tw = reinterpret_cast<float*>(Rs) + (warp & 3) * (32 * 36);       // [32 heads][36 floats]
    float* ph_warp = a.partials + (((long long)i * a.Hq + hb * HBLK + 32 * (warp & 3)) * a.nsplit + sp) * PSM;
#pragma unroll 1
    for (int c = 0; c < DVH / 32; ++c) {
      uint32_t o[32];
      if (have) {
        tmem_ld32_issue(lane_addr + COL_O + 32 * c, o);
        tmem_ld_wait(o);
      } else {
#pragma unroll
        for (int e = 0; e < 32; ++e) o[e] = 0u;
      }
#pragma unroll
      for (int e = 0; e < 8; ++e)
        *reinterpret_cast<uint4*>(tw + lane * 36 + 4 * e) = make_uint4(o[4 * e], o[4 * e + 1], o[4 * e + 2], o[4 * e + 3]);
      __syncwarp();
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int r = 4 * k + (lane >> 3), piece = lane & 7;
        const uint4 v = *reinterpret_cast<const uint4*>(tw + r * 36 + 4 * piece);
        *reinterpret_cast<uint4*>(ph_warp + (long long)r * a.nsplit * PSM + 4 + hd * DVH + 32 * c + 4 * piece) = v;
      }
      __syncwarp();
    }
  }

  fence_before();
  __syncthreads();
  fence_after();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  if (tid == 0 && *abort_flag && a.status) atomicOr(a.status, SNAP_DEV_WAIT_TIMEOUT);
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

size_t stream_smem_bytes() { return (size_t)NSLAB * QSLAB_B + NSTG * STAGE_B + (2 * NSTG + 7) * 8 + 16 + 1024; }

}  // namespace

bool decode_mla_stream_supported(int dtype, const Shape& s) {
  return dtype == SNAP_BF16 && s.v_aliases_k && s.d_qk == DQK && s.d_v == DV && s.Hkv == 1 && s.Hq % HBLK == 0 &&
         umma::encode_tiled_fn() != nullptr;
}

// Row splits per sequence: the grid (splits x 2 value halves x head blocks x sequences) should
// fill the SMs once or twice over, with at least two tiles per split.
int decode_mla_stream_nsplit(const Shape& s, int n_active, int sm_count) {
  const int tiles = (s.Sc + TR - 1) / TR + 1;
  if (const int v = option(SNAP_OPT_DECODE_NSPLIT)) return v < tiles ? (v < 64 ? v : 64) : tiles;   // tuning aid
  const long long base = (long long)n_active * NHALF * (s.Hq / HBLK);
  int best = 1;
  double best_fill = -1.0;
  for (int ns = 1; ns <= 64 && ns <= (tiles / 2 > 1 ? tiles / 2 : 1); ++ns) {
    const long long ctas = base * ns;
    const long long waves = (ctas + sm_count - 1) / sm_count;
    if (waves > 2 && ns > 1) break;
    const double fill = (double)ctas / (double)(waves * sm_count);
    if (fill > best_fill + 1e-9) { best_fill = fill; best = ns; }
  }
  return best;
}

size_t decode_mla_stream_partial_floats(const Shape& s, int n_active, int nsplit) {
  return (size_t)n_active * s.Hq * nsplit * PSM;
}

cudaError_t launch_decode_mla_stream(const Shape& s, const void* q, const void* k_new, const int* slot_ids,
                                     int n_active, void* k_cache, int* seq_len, const int* valid_topk, void* out,
                                     float* partials, int nsplit, uint32_t* status, cudaStream_t st, int q_len, int u) {
  if (n_active == 0) return cudaSuccess;
  umma::EncodeTiledFn enc = umma::encode_tiled_fn();
  if (!enc) return cudaErrorNotSupported;
  CUtensorMap tq, tk, tv;
  const cuuint32_t estr3[3] = {1, 1, 1};
  {
    // queries [n_active][q_len][Hq][576]: token u of every sequence as a (dim, head, sequence) tensor
    const cuuint64_t dims[3] = {(cuuint64_t)DQK, (cuuint64_t)s.Hq, (cuuint64_t)n_active};
    const cuuint64_t strides[2] = {(cuuint64_t)DQK * 2, (cuuint64_t)q_len * s.Hq * DQK * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)HBLK, 1};
    void* q_u = const_cast<__nv_bfloat16*>(static_cast<const __nv_bfloat16*>(q) + (long long)u * s.Hq * DQK);
    if (enc(&tq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, q_u, dims, strides, box, estr3,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
  }
  const cuuint64_t dims[3] = {(cuuint64_t)DQK, (cuuint64_t)s.Sc, (cuuint64_t)s.max_seqs};
  const cuuint64_t strides[2] = {(cuuint64_t)DQK * 2, (cuuint64_t)s.Sc * DQK * 2};
  const cuuint32_t kbox[3] = {64, (cuuint32_t)TR, 1}, vbox[3] = {64, (cuuint32_t)VROWS, 1};
  if (enc(&tk, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, k_cache, dims, strides, kbox, estr3, CU_TENSOR_MAP_INTERLEAVE_NONE,
          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
      enc(&tv, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, k_cache, dims, strides, vbox, estr3, CU_TENSOR_MAP_INTERLEAVE_NONE,
          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  SArgs a;
  a.k_new = k_new ? static_cast<const __nv_bfloat16*>(k_new) + (long long)u * DQK : nullptr;   // Hkv = 1
  a.knew_seq_stride = (long long)q_len * DQK;
  a.kc = static_cast<unsigned char*>(k_cache);
  a.slot_ids = slot_ids; a.seq_len = seq_len; a.valid_topk = valid_topk;
  a.Hq = s.Hq; a.Ls = s.Ls; a.Lr = s.Lr; a.Sc = s.Sc; a.max_seqs = s.max_seqs; a.nsplit = nsplit;
  a.scale_log2 = s.scale * 1.4426950408889634f;
  a.partials = partials; a.status = status;
  const size_t smem = stream_smem_bytes();
  static SmemLimit limit = {};
  if (cudaError_t e = ensure_dyn_smem(decode_mla_stream_kernel, smem, limit)) return e;
  // a programmatic dependent launch: the CTAs may become resident while the previous kernel drains
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(nsplit, NHALF * (s.Hq / HBLK), n_active);
  lc.blockDim = dim3(NTH);
  lc.dynamicSmemBytes = smem;
  lc.stream = st;
  lc.attrs = attr;
  lc.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&lc, decode_mla_stream_kernel, a, tq, tk, tv);
  count_launch();
  if (e != cudaSuccess) return e;
  return launch_decode_mla_merge(partials, out, n_active, s.Hq, nsplit, slot_ids, seq_len, s.max_seqs, k_new != nullptr, st, true,
                                 q_len, u);
}

}  // namespace snap
