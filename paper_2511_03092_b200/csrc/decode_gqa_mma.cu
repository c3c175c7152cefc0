// Decode attention over the compressed cache (Section 3.3) for bf16 layers with 64-, 128- or 256-wide
// heads and 1 to 16 query heads per KV head, on tensor cores -- the HBM-bound kernel of the decode step.
//
// Split-K flash decoding: grid = splits x KV heads x sequences, warp-private pipelines of 16-row
// tiles, one partial result per split, a merge kernel.  The arithmetic is mma.sync.m16n8k16
// with the group's heads on the N side:
//     S^T[16 rows x 8 columns]   = K tile [16 x 128] . Q^T                    (8 MMAs)
//     O^T[128 dims x 8 columns] += V tile^T [128 x 16] . P^T [16 x 8 columns] (8 MMAs)
// so the cost per cache row does not depend on the group size (with packed FP32 arithmetic the
// multiply-adds outrun the FP32 pipe from five heads per KV head on, and cost issue slots
// before that).  Tiles arrive through TMA tensor loads with the 128-byte swizzle (two 64-dim
// slabs per tensor, per-warp mbarriers), which makes the ldmatrix reads conflict-free; V is read
// with ldmatrix.trans; the probabilities leave the S^T accumulators for the B operand of the
// second product through movmatrix (an 8x8 transpose across the warp).  Online softmax is per
// column in the log2 domain with a lazily refreshed reference; row sums are kept per thread
// and reduced once at the end.
//
// Fused append (Eq. 3): the warp that stages the new token's slot stores the row to the cache
// and patches its staged copy.
//
// Several new tokens per step (multi-token prediction): the columns are then (token, head)
// pairs: T x g <= 8 in the usual instantiation, up to 16 in a second one (NG = 2: two groups of
// eight columns, i.e. two MMAs per fragment of K or V, for steps of three or four tokens at g = 4).  Query t must see the cache as it is after tokens 0..t: the old rows
// are attended as staged, a window row that token u evicts is masked for the queries from u
// on, the new rows form one extra tile with a causal mask, and each new row is written to the
// cache by the warp that has just staged the row it replaces.
#include <cuda.h>

#include "mma_helpers.cuh"
#include "snap_internal.cuh"
#include "umma_helpers.cuh"

namespace snap {
namespace {

using namespace mmasync;

using umma::mbar_init;
using umma::mbar_expect_tx;
using umma::mbar_try_wait;
using umma::smem_u32;
using umma::tma_load_3d;

constexpr int WT = 16, NSTAGE = 2, GP = 8;     // 16-row tiles, two stages per warp, GP: column slots (N of the MMAs)
constexpr int SLAB_B = WT * 128;                // one 64-dim slab of a tile: 16 rows x 128 bytes
constexpr unsigned kWaitLimit = 1u << 22;

struct MmaArgs {
  const __nv_bfloat16* q; const __nv_bfloat16* k_new; const __nv_bfloat16* v_new;
  const int* slot_ids;
  char* kc; char* vc;
  long long seq_b, head_b;
  int Hq, Hkv, g, Ls, Lr, max_seqs, nsplit;
  int T;                                        // query tokens per sequence in this launch (T * g <= 16)
  int QT, u0;                                   // ... which are tokens u0 .. u0 + T - 1 of the QT tokens per sequence in q / k_new / v_new
  float scale_log2;
  const int* seq_len; const int* valid_topk;
  float* partials;                              // [n_active][T][Hq][nsplit][PS]
  __nv_bfloat16* out;                           // fused merge only: [n_active][QT][Hq][D]
  uint32_t* status;
  // per-step block lookup (block_topk.cu): NULL, or the blocks of the third section to visit, ascending
  const int* block_idx;                         // [n_active][Hkv][blocks_cap]
  const int* n_sel;                             // [n_active][Hkv] entries of block_idx in use
  int blocks_cap, tpb;                          // tiles per block = block_tokens / 16
};

__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, unsigned parity) {
  for (unsigned it = 0; it < kWaitLimit; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
// byte offset of row r, 16-byte chunk c (0..7) inside a 128-byte-swizzled slab
__device__ __forceinline__ uint32_t swz(int r, int c) { return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4)); }

// Tile j of a (sequence, KV head): cache rows [row0, row0 + WT), valid below row_end.  Tiles
// cover [0, n_low) first, then [Lsr, Lsr + n_top); a tile never spans the two regions.
struct TileRows { int row0, row_end; };
__device__ __forceinline__ TileRows tile_rows(int j, int nA, int n_low, int Lsr, int n_top) {
  TileRows t;
  if (j < nA) { t.row0 = j * WT; t.row_end = n_low; }
  else { t.row0 = Lsr + (j - nA) * WT; t.row_end = Lsr + n_top; }
  return t;
}

// D: head size (64, 128 or 256); NWARP: warps per CTA (fewer for wide heads, whose stages are larger);
// NG: groups of eight MMA columns (1, or 2 for multi-token steps with 9 to 16 query rows per KV head)
// FUSED: the splits of a (sequence, KV head) form one thread-block cluster (the grid's x extent) and merge
// their results through distributed shared memory instead of a second launch -- for small batches, where a
// step is a chain of launch latencies.  Every CTA reduces an equal share of the output elements: each split
// sends every CTA that CTA's share of its outputs, and its (max, sum) per column, with asynchronous remote
// stores that complete on the receiver's mbarrier; a CTA waits for its own arrivals only, so the one cluster
// barrier (the mbarriers exist before anything is sent) is started at the top of the kernel and completed
// just before the sends, and none is needed at the end.
template <int D, int NWARP, int NG, bool FUSED>
__global__ void __launch_bounds__(NWARP * 32, NG == 1 ? 3 : 2)
decode_gqa_mma_kernel(const MmaArgs a, const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v) {
  constexpr int NT = NWARP * 32, NSL = D / 64, CPR = D / 8, KS = D / 16;   // slabs per tensor, 16-byte chunks per row, 16-dim steps
  constexpr int TENS_B = NSL * SLAB_B, STAGE_B = 2 * TENS_B, PS = D + 2;   // stage = K slabs | V slabs
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem_raw = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  // [NWARP][NSTAGE] stages | [NWARP][NSTAGE] mbarriers
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_raw + NWARP * NSTAGE * STAGE_B);
  // fused merge: this split's outputs [columns][D] (+ padding), its (max, sum) per column, the inbox
  // [splits][share of the outputs + 16] and the inbox's barrier
  constexpr int XO = NG * GP * D + 64;
  float* osm = reinterpret_cast<float*>(bars + NWARP * NSTAGE);
  float* mls = osm + XO;
  float* inbox = mls + 16;
  uint64_t* xbar = reinterpret_cast<uint64_t*>(inbox + XO + 16 * 16);

  const int sp = blockIdx.x, kvh = blockIdx.y, i = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5, gq = lane >> 2, tq = lane & 3;
  unsigned char* wstages = smem_raw + w * NSTAGE * STAGE_B;
  const uint32_t stage0 = smem_u32(wstages), bar0 = smem_u32(bars + w * NSTAGE);
  if (lane == 0) {
    for (int s = 0; s < NSTAGE; ++s) mbar_init(bar0 + 8 * s, 1);
    if (FUSED && tid == 0) mbar_init(smem_u32(xbar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  if (FUSED) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");   // completed before the merge's sends
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int slot = a.slot_ids[i];
  const bool bad = slot < 0 || slot >= a.max_seqs;
  const int Lsr = a.Ls + a.Lr, TQ = a.T;
  // One new token (the usual step): its row is patched into the staged tile, so it counts as valid.
  // Several new tokens: query t must see the cache as it is after tokens 0..t, so the old rows
  // are attended as they are (the rows that tokens evict masked per query) and the new rows
  // form a tile of their own; n_low_st then only extends the tile list to the slots they fill.
  int L0 = 0, n_low = 0, n_low_st = 0, n_top = 0, new_slot = -1;
  if (!bad) {
    L0 = a.seq_len[slot];
    n_top = a.valid_topk[slot];
    if (TQ == 1) {
      n_low = n_low_st = min(L0 + (a.k_new ? 1 : 0), Lsr);
      if (a.k_new) new_slot = ring_slot(L0, a.Ls, a.Lr);
    } else {
      n_low = min(L0, Lsr);
      n_low_st = min(L0 + TQ, Lsr);
    }
  } else if (tid == 0 && sp == 0 && kvh == 0 && a.status) {
    atomicOr(a.status, SNAP_DEV_BAD_SLOT);
  }
  const int* blist = a.block_idx && !bad ? a.block_idx + ((long long)i * a.Hkv + kvh) * a.blocks_cap : nullptr;
  const int nA = (n_low_st + WT - 1) / WT;
  const int ntiles = nA + (blist ? a.n_sel[i * a.Hkv + kvh] * a.tpb : (n_top + WT - 1) / WT);
  // tile j: the low section first, then the third section -- all of it, or the listed blocks only
  auto rows_of = [&](int j) -> TileRows {
    if (j < nA || !blist) return tile_rows(j, nA, n_low, Lsr, n_top);
    const int jj = j - nA, blk = blist[jj / a.tpb];
    TileRows t;
    t.row0 = Lsr + (blk * a.tpb + jj % a.tpb) * WT;
    t.row_end = Lsr + n_top;
    return t;
  };
  const int t_begin = (int)((long long)ntiles * sp / a.nsplit);
  const int t_end = (int)((long long)ntiles * (sp + 1) / a.nsplit);
  // this warp's tiles: t_begin + w, t_begin + w + NWARP, ...
  const int T = t_end - t_begin > w ? (t_end - t_begin - w + NWARP - 1) / NWARP : 0;
  const int plane = bad ? 0 : slot * a.Hkv + kvh;               // third tensor-map coordinate

  auto issue = [&](int n) {                                     // tile n of this warp -> stage n % NSTAGE
    const int s = n % NSTAGE;
    const TileRows tr = rows_of(t_begin + w + n * NWARP);
    const uint32_t dst = stage0 + s * STAGE_B, bar = bar0 + 8 * s;
    mbar_expect_tx(bar, (unsigned)STAGE_B);
#pragma unroll
    for (int h = 0; h < NSL; ++h) {
      tma_load_3d(dst + h * SLAB_B, &tmap_k, 64 * h, tr.row0, plane, bar);
      tma_load_3d(dst + TENS_B + h * SLAB_B, &tmap_v, 64 * h, tr.row0, plane, bar);
    }
  };
  if (lane == 0)
    for (int n = 0; n < NSTAGE && n < T; ++n) issue(n);

  char* kc = a.kc + slot * a.seq_b + kvh * a.head_b;
  char* vc = a.vc + slot * a.seq_b + kvh * a.head_b;
  // new rows of this KV head: token u at kn + u * Hkv * D
  const __nv_bfloat16* kn = a.k_new ? a.k_new + (((long long)i * a.QT + a.u0) * a.Hkv + kvh) * D : nullptr;
  const __nv_bfloat16* vn = a.v_new ? a.v_new + (((long long)i * a.QT + a.u0) * a.Hkv + kvh) * D : nullptr;
  const long long new_stride = (long long)a.Hkv * D;

  // Column n of the MMAs is query token n / g, head n % g of the group (zero beyond T * g).
  // B fragments of Q^T for the eight 16-dim steps: column gq, dims 16 ks + 2 tq (+8)
  const int ncols = TQ * a.g;
  uint32_t qb[NG][KS][2];
  int tc0[NG], tc1[NG];                          // query tokens of this thread's two columns, per column group
#pragma unroll
  for (int gi = 0; gi < NG; ++gi) {
    const int col = GP * gi + gq;                // this lane's column of the B fragments
    const int tcol = col / a.g, hcol = col - tcol * a.g;
    const __nv_bfloat16* qp = a.q + (((long long)i * a.QT + a.u0 + tcol) * a.Hq + (long long)kvh * a.g + hcol) * D + 2 * tq;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qb[gi][ks][0] = col < ncols ? *reinterpret_cast<const uint32_t*>(qp + 16 * ks) : 0u;
      qb[gi][ks][1] = col < ncols ? *reinterpret_cast<const uint32_t*>(qp + 16 * ks + 8) : 0u;
    }
    tc0[gi] = (GP * gi + 2 * tq) / a.g;
    tc1[gi] = (GP * gi + 2 * tq + 1) / a.g;
  }
  float oacc[NG][KS][4];                         // O^T: dims 16 db + gq (+8), columns 8 gi + 2 tq (+1)
#pragma unroll
  for (int gi = 0; gi < NG; ++gi)
#pragma unroll
    for (int db = 0; db < KS; ++db)
#pragma unroll
      for (int e = 0; e < 4; ++e) oacc[gi][db][e] = 0.f;
  float m_ref[NG][2], l_part[NG][2];             // columns 8 gi + 2 tq, 8 gi + 2 tq + 1
#pragma unroll
  for (int gi = 0; gi < NG; ++gi) { m_ref[gi][0] = m_ref[gi][1] = -INFINITY; l_part[gi][0] = l_part[gi][1] = 0.f; }
  bool timed_out = false;

  // ldmatrix lane roles: K (plain): row (lane & 7) + 8 * bit3, chunk + bit4; V (transposed): row (lane & 7) + 8 * bit4, chunk + bit3
  const int k_row = (lane & 7) + ((lane >> 3) & 1) * 8, k_cadd = lane >> 4;
  const int v_row = (lane & 7) + ((lane >> 4) & 1) * 8, v_cadd = (lane >> 3) & 1;

  // One staged tile: ok[gi][N] says whether this thread's value N of column group gi (rows gq, gq, gq + 8,
  // gq + 8 x columns 2 tq, 2 tq + 1, 2 tq, 2 tq + 1) takes part.
  struct Mask { bool ok[NG][4]; };
  auto process = [&](uint32_t sK, uint32_t sV, const Mask& mk) {
    // ---- S^T = K tile . Q^T ----
    float sacc[NG][4];
#pragma unroll
    for (int gi = 0; gi < NG; ++gi) { sacc[gi][0] = sacc[gi][1] = sacc[gi][2] = sacc[gi][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      uint32_t af[4];
      ldsm4(sK + (ks >> 2) * SLAB_B + swz(k_row, (ks & 3) * 2 + k_cadd), af);
#pragma unroll
      for (int gi = 0; gi < NG; ++gi) mma16816(sacc[gi], af, qb[gi][ks][0], qb[gi][ks][1]);
    }
    float v[NG][4];
    bool refresh = false;
#pragma unroll
    for (int gi = 0; gi < NG; ++gi) {
#pragma unroll
      for (int e = 0; e < 4; ++e) v[gi][e] = mk.ok[gi][e] ? sacc[gi][e] * a.scale_log2 : -INFINITY;
      refresh = refresh || fmaxf(v[gi][0], v[gi][2]) > m_ref[gi][0] + 8.f || fmaxf(v[gi][1], v[gi][3]) > m_ref[gi][1] + 8.f;
    }
    // Lazy reference per column: refreshed (accumulators rescaled) only when a warp vote sees a
    // logit 8 above it; the column maxima are then reduced over the lanes that share tq.
    if (__any_sync(0xffffffffu, refresh)) {
#pragma unroll
      for (int gi = 0; gi < NG; ++gi) {
        float mx0 = fmaxf(v[gi][0], v[gi][2]), mx1 = fmaxf(v[gi][1], v[gi][3]);
#pragma unroll
        for (int o = 4; o <= 16; o <<= 1) {
          mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, o));
          mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, o));
        }
        const float n0 = fmaxf(m_ref[gi][0], mx0), n1 = fmaxf(m_ref[gi][1], mx1);
        const float a0 = m_ref[gi][0] == -INFINITY ? 0.f : exp2f(m_ref[gi][0] - n0);
        const float a1 = m_ref[gi][1] == -INFINITY ? 0.f : exp2f(m_ref[gi][1] - n1);
        m_ref[gi][0] = n0; m_ref[gi][1] = n1;
        l_part[gi][0] *= a0; l_part[gi][1] *= a1;
#pragma unroll
        for (int db = 0; db < KS; ++db) {
          oacc[gi][db][0] *= a0; oacc[gi][db][1] *= a1; oacc[gi][db][2] *= a0; oacc[gi][db][3] *= a1;
        }
      }
    }
    uint32_t pb[NG][2];
#pragma unroll
    for (int gi = 0; gi < NG; ++gi) {
      const float r0 = m_ref[gi][0] == -INFINITY ? 0.f : m_ref[gi][0], r1 = m_ref[gi][1] == -INFINITY ? 0.f : m_ref[gi][1];
      const float p0 = fast_exp2(v[gi][0] - r0), p1 = fast_exp2(v[gi][1] - r1);
      const float p2 = fast_exp2(v[gi][2] - r0), p3 = fast_exp2(v[gi][3] - r1);
      l_part[gi][0] += p0 + p2;
      l_part[gi][1] += p1 + p3;
      // P^T as the B operand: rows 2 tq (+1) and 2 tq + 8 (+9) of column gq
      pb[gi][0] = movmatrix_t(pack_bf16(p0, p1));
      pb[gi][1] = movmatrix_t(pack_bf16(p2, p3));
    }
    // ---- O^T += V tile^T . P^T ----
#pragma unroll
    for (int db = 0; db < KS; ++db) {
      uint32_t af[4];
      ldsm4t(sV + (db >> 2) * SLAB_B + swz(v_row, (db & 3) * 2 + v_cadd), af);
#pragma unroll
      for (int gi = 0; gi < NG; ++gi) mma16816(oacc[gi][db], af, pb[gi][0], pb[gi][1]);
    }
  };

  for (int n = 0; n < T; ++n) {
    const int s = n % NSTAGE;
    const unsigned parity = (unsigned)(n / NSTAGE) & 1u;
    const bool landed = mbar_wait_bounded(bar0 + 8 * s, parity);
    if (__any_sync(0xffffffffu, !landed)) { timed_out = true; break; }
    const int j = t_begin + w + n * NWARP;
    const TileRows tr = rows_of(j);
    const int nrows = tr.row_end - tr.row0;                    // rows at or past it are masked (may be <= 0)
    const uint32_t sK = stage0 + s * STAGE_B, sV = sK + TENS_B;
    Mask mk;
#pragma unroll
    for (int gi = 0; gi < NG; ++gi) { mk.ok[gi][0] = mk.ok[gi][1] = gq < nrows; mk.ok[gi][2] = mk.ok[gi][3] = gq + 8 < nrows; }
    if (nrows < WT) {
      // ragged tile: rows past the end may hold anything (memory the caller never wrote), and a
      // zero probability does not silence a NaN in V: clear those V rows
      const int first = max(nrows, 0);
      for (int e = lane; e < (WT - first) * CPR; e += 32) {
        const int r = first + e / CPR, c = e % CPR;
        *reinterpret_cast<uint4*>(wstages + s * STAGE_B + TENS_B + (c >> 3) * SLAB_B + swz(r, c & 7)) = make_uint4(0, 0, 0, 0);
      }
      __syncwarp();
    }
    if (TQ == 1) {
      if (new_slot >= tr.row0 && new_slot < tr.row0 + WT && new_slot < tr.row_end) {
        // the new token's slot is in this tile: store the row to the cache and patch the staged copy
        const int r = new_slot - tr.row0;
        for (int e = lane; e < 2 * CPR; e += 32) {             // K chunks, then V chunks of the row
          const int tens = e / CPR, c = e % CPR;
          const uint4 val = reinterpret_cast<const uint4*>(tens ? vn : kn)[c];
          reinterpret_cast<uint4*>((tens ? vc : kc) + (long long)new_slot * (D * 2))[c] = val;
          *reinterpret_cast<uint4*>(wstages + s * STAGE_B + tens * TENS_B + (c >> 3) * SLAB_B + swz(r, c & 7)) = val;
        }
        __syncwarp();
      }
    } else if (j < nA) {
      // new tokens whose slot lies in this tile: the old row (if the token evicts one) stays visible to
      // the queries before that token only; the new row goes to the cache now that the old one is staged
      for (int u = 0; u < TQ; ++u) {
        const int ru = ring_slot(L0 + u, a.Ls, a.Lr);
        if (ru < tr.row0 || ru >= tr.row0 + WT) continue;
        const int r = ru - tr.row0;
#pragma unroll
        for (int gi = 0; gi < NG; ++gi) {
          if (gq == r) { mk.ok[gi][0] = mk.ok[gi][0] && tc0[gi] < u; mk.ok[gi][1] = mk.ok[gi][1] && tc1[gi] < u; }
          if (gq + 8 == r) { mk.ok[gi][2] = mk.ok[gi][2] && tc0[gi] < u; mk.ok[gi][3] = mk.ok[gi][3] && tc1[gi] < u; }
        }
        for (int e = lane; e < 2 * CPR; e += 32) {
          const int tens = e / CPR, c = e % CPR;
          reinterpret_cast<uint4*>((tens ? vc : kc) + (long long)ru * (D * 2))[c] =
              reinterpret_cast<const uint4*>((tens ? vn : kn) + u * new_stride)[c];
        }
      }
    }
    process(sK, sV, mk);
    __syncwarp();
    if (lane == 0 && n + NSTAGE < T) {
      // the stage was read, and possibly patched, through the generic proxy; the bulk copy that
      // refills it goes through the async proxy
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      issue(n + NSTAGE);
    }
  }
  if (timed_out) {
    if (a.status) atomicOr(a.status, SNAP_DEV_WAIT_TIMEOUT);
    for (int s = 0; s < NSTAGE; ++s) (void)mbar_wait_bounded(bar0 + 8 * s, 0u);
  }
  if (TQ > 1 && sp == 0 && w == 0 && !bad && !timed_out) {
    // the new tokens as a tile of their own (this warp's pipeline has drained): row u is token u,
    // visible to the queries from token u on; rows past the last token are zero and masked
    for (int e = lane; e < 2 * WT * CPR; e += 32) {
      const int tens = e / (WT * CPR), r = (e / CPR) % WT, c = e % CPR;
      uint4 val = make_uint4(0, 0, 0, 0);
      if (r < TQ) val = reinterpret_cast<const uint4*>((tens ? vn : kn) + r * new_stride)[c];
      *reinterpret_cast<uint4*>(wstages + tens * TENS_B + (c >> 3) * SLAB_B + swz(r, c & 7)) = val;
    }
    __syncwarp();
    Mask mk;
#pragma unroll
    for (int gi = 0; gi < NG; ++gi) {
      mk.ok[gi][0] = gq < TQ && gq <= tc0[gi]; mk.ok[gi][1] = gq < TQ && gq <= tc1[gi];
      mk.ok[gi][2] = gq + 8 < TQ && gq + 8 <= tc0[gi]; mk.ok[gi][3] = gq + 8 < TQ && gq + 8 <= tc1[gi];   // up to 16 tokens
    }
    process(stage0, stage0 + TENS_B, mk);
    __syncwarp();
  }

  // ---- per-warp result -> this warp's stage memory, then merge the warps ----
  constexpr int NCOL = NG * GP;
  float* wm = reinterpret_cast<float*>(wstages);           // [NCOL] max, [NCOL] sum, [NCOL][D] acc
  float* wl = wm + NCOL;
  float* wacc = wl + NCOL;
  __syncwarp();
#pragma unroll
  for (int gi = 0; gi < NG; ++gi) {
#pragma unroll
    for (int o = 4; o <= 16; o <<= 1) {
      l_part[gi][0] += __shfl_xor_sync(0xffffffffu, l_part[gi][0], o);
      l_part[gi][1] += __shfl_xor_sync(0xffffffffu, l_part[gi][1], o);
    }
    const int c0 = GP * gi + 2 * tq;
    if (gq == 0) {
      wm[c0] = m_ref[gi][0]; wm[c0 + 1] = m_ref[gi][1];
      wl[c0] = l_part[gi][0]; wl[c0 + 1] = l_part[gi][1];
    }
#pragma unroll
    for (int db = 0; db < KS; ++db) {
      wacc[c0 * D + 16 * db + gq] = oacc[gi][db][0];
      wacc[(c0 + 1) * D + 16 * db + gq] = oacc[gi][db][1];
      wacc[c0 * D + 16 * db + gq + 8] = oacc[gi][db][2];
      wacc[(c0 + 1) * D + 16 * db + gq + 8] = oacc[gi][db][3];
    }
  }
  __syncthreads();
  constexpr int WSTRIDE = NSTAGE * STAGE_B / 4;            // floats between two warps' regions
  const float* base = reinterpret_cast<const float*>(smem_raw);
  for (int h = 0; h < ncols; ++h) {
    float M = -INFINITY;
#pragma unroll
    for (int ww = 0; ww < NWARP; ++ww) M = fmaxf(M, base[ww * WSTRIDE + h]);
    float L = 0.f, f[NWARP];
#pragma unroll
    for (int ww = 0; ww < NWARP; ++ww) {
      const float mw = base[ww * WSTRIDE + h];
      f[ww] = mw == -INFINITY ? 0.f : exp2f(mw - M);
      L += base[ww * WSTRIDE + NCOL + h] * f[ww];
    }
    const int tcol = h / a.g, hcol = h - tcol * a.g;
    // this split's result for column h: to scratch for the merge kernel, or to this CTA's exchange area
    float* ph = a.partials + ((((long long)i * TQ + tcol) * a.Hq + (long long)kvh * a.g + hcol) * a.nsplit + sp) * PS;
    if (tid == 0) {
      if (FUSED) { mls[2 * h] = M; mls[2 * h + 1] = L; }
      else { ph[0] = M; ph[1] = L; }
    }
    for (int dv = tid; dv < D; dv += NT) {
      float O = 0.f;
#pragma unroll
      for (int ww = 0; ww < NWARP; ++ww) O += base[ww * WSTRIDE + 2 * NCOL + h * D + dv] * f[ww];
      if (FUSED) osm[h * D + dv] = O;
      else ph[2 + dv] = O;
    }
  }
  if (FUSED) {
    const int ns = a.nsplit;                                   // = cluster size; sp = this CTA's rank in the cluster
    const int W = ncols * D;
    const int per = (((W + ns - 1) / ns) + 3) & ~3;            // outputs reduced by each CTA, whole 16-byte pieces
    const int pp = per / 4 + 4, row = per + 16;                // pieces sent to each CTA: its outputs, then 16 floats of (max, sum)
    __syncthreads();                                           // osm and mls are complete
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");   // every CTA's inbox barrier exists
    if (tid == 0) mbar_expect_tx(smem_u32(xbar), (unsigned)(ns * pp * 16));
    const uint32_t my_row = smem_u32(inbox) + (uint32_t)(sp * row) * 4u, xb = smem_u32(xbar);
    for (int e = tid; e < ns * pp; e += NT) {
      const int to = e / pp, piece = e - to * pp;
      const float* src = piece < per / 4 ? osm + to * per + 4 * piece : mls + 4 * (piece - per / 4);
      const uint4 v = *reinterpret_cast<const uint4*>(src);
      asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
                   ::"r"(umma::map_to_rank(my_row + (uint32_t)piece * 16u, (uint32_t)to)), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w),
                     "r"(umma::map_to_rank(xb, (uint32_t)to)) : "memory");
    }
    if (!mbar_wait_bounded(smem_u32(xbar), 0u)) {
      if (tid == 0 && a.status) atomicOr(a.status, SNAP_DEV_WAIT_TIMEOUT);
    } else {
      for (int ol = tid; ol < per; ol += NT) {
        const int o = sp * per + ol;
        if (o >= W) break;
        const int h = o / D, dv = o - h * D;
        float M = -INFINITY;
        for (int rr = 0; rr < ns; ++rr) M = fmaxf(M, inbox[rr * row + per + 2 * h]);
        float L = 0.f, O = 0.f;
        for (int rr = 0; rr < ns; ++rr) {
          const float mr = inbox[rr * row + per + 2 * h];
          const float fr = mr == -INFINITY ? 0.f : exp2f(mr - M);
          L = fmaf(inbox[rr * row + per + 2 * h + 1], fr, L);
          O = fmaf(inbox[rr * row + ol], fr, O);
        }
        const int tcol = h / a.g, hcol = h - tcol * a.g;
        const long long orow = (long long)i * a.QT + a.u0 + tcol;
        a.out[(orow * a.Hq + (long long)kvh * a.g + hcol) * D + dv] = __float2bfloat16_rn(L > 0.f ? O / L : 0.f);
      }
    }
  }
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// The sequence lengths advance after every CTA of the step has read them: with the fused merge that is a
// launch of its own (a few threads), off the path of the step's outputs.
__global__ void decode_gqa_bump_kernel(const int* __restrict__ slot_ids, int* seq_len, int max_seqs, int n_rows, int q_len) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r < n_rows) {
    const int slot = slot_ids[r / q_len];
    if (slot >= 0 && slot < max_seqs) atomicAdd(&seq_len[slot], 1);
  }
}

// Merge the splits of one (sequence, query token, query head) for any head size; maxima are in
// the log2 domain.  Rows of `partials` are indexed by sequence * q_len + token; the token is token
// u0 + (its index) of the q_total per sequence in `out`; every token's block advances the sequence
// length by one.
__global__ void __launch_bounds__(128) decode_gqa_mma_merge_kernel(const float* __restrict__ partials,
                                                                   __nv_bfloat16* __restrict__ out, int Hq, int d,
                                                                   int nsplit, const int* __restrict__ slot_ids,
                                                                   int* seq_len, int max_seqs, int bump, int q_len, int q_total,
                                                                   int u0) {
  const int h = blockIdx.x, i = blockIdx.y, ps = d + 2;
  const long long orow = (long long)(i / q_len) * q_total + u0 + i % q_len;   // token's row of `out`
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const float* p = partials + ((long long)i * Hq + h) * nsplit * ps;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  float M = -INFINITY, L = 0.f;
  if (nsplit <= 128) {                                       // (m, l) fetched by one thread per split, weights in shared memory
    __shared__ float m_s[128], l_s[128], f_s[128];
    const int t0 = threadIdx.x;
    if (t0 < nsplit) { m_s[t0] = p[t0 * ps]; l_s[t0] = p[t0 * ps + 1]; }
    __syncthreads();
    for (int s = 0; s < nsplit; ++s) M = fmaxf(M, m_s[s]);
    if (t0 < nsplit) f_s[t0] = m_s[t0] == -INFINITY ? 0.f : exp2f(m_s[t0] - M);
    __syncthreads();
    for (int s = 0; s < nsplit; ++s) L += l_s[s] * f_s[s];
    const float inv = L > 0.f ? 1.f / L : 0.f;
    for (int t = threadIdx.x; t < d; t += blockDim.x) {
      float O = 0.f;
#pragma unroll 8
      for (int s = 0; s < nsplit; ++s) O = fmaf(p[s * ps + 2 + t], f_s[s], O);
      out[(orow * Hq + h) * d + t] = __float2bfloat16_rn(O * inv);
    }
  } else {
    for (int s = 0; s < nsplit; ++s) M = fmaxf(M, p[s * ps]);
    for (int s = 0; s < nsplit; ++s) {
      const float ms = p[s * ps];
      if (ms != -INFINITY) L += p[s * ps + 1] * exp2f(ms - M);
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
    for (int t = threadIdx.x; t < d; t += blockDim.x) {
      float O = 0.f;
      for (int s = 0; s < nsplit; ++s) {
        const float ms = p[s * ps];
        if (ms != -INFINITY) O += p[s * ps + 2 + t] * exp2f(ms - M);
      }
      out[(orow * Hq + h) * d + t] = __float2bfloat16_rn(O * inv);
    }
  }
  if (bump && h == 0 && threadIdx.x == 0) {
    const int slot = slot_ids[i / q_len];
    if (slot >= 0 && slot < max_seqs) atomicAdd(&seq_len[slot], 1);
  }
}

template <int D, int NWARP, int NG, bool FUSED>
cudaError_t launch_d(const MmaArgs& a, const CUtensorMap& tk, const CUtensorMap& tv, int n_active, cudaStream_t st) {
  constexpr size_t smem = (size_t)NWARP * NSTAGE * (2 * (D / 64) * SLAB_B) + NWARP * NSTAGE * 8 + 1024 +
                          (FUSED ? (size_t)(2 * (NG * GP * D + 64) + 16 + 16 * 16) * sizeof(float) + 16 : 0);
  static_assert((size_t)NSTAGE * (2 * (D / 64) * SLAB_B) >= (size_t)NG * GP * (D + 2) * sizeof(float), "a warp's result fits its stages");
  static SmemLimit limit = {};
  if (cudaError_t e = ensure_dyn_smem(decode_gqa_mma_kernel<D, NWARP, NG, FUSED>, smem, limit)) return e;
  cudaError_t e;
  if (FUSED) {
    // the splits of a (sequence, KV head) as one cluster; more than eight CTAs per cluster need the opt-in
    static bool allowed = false;
    if (a.nsplit > 8 && !allowed) {
      if ((e = cudaFuncSetAttribute(decode_gqa_mma_kernel<D, NWARP, NG, FUSED>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1)) != cudaSuccess)
        return e;
      allowed = true;
    }
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)a.nsplit;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(a.nsplit, a.Hkv, n_active);
    lc.blockDim = dim3(NWARP * 32);
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    lc.attrs = attr;
    lc.numAttrs = 2;
    // can the device hold a cluster of this size at all?  Asked once per size, before the launch: a launch that
    // fails inside a stream capture would invalidate the caller's capture.
    static int fits[17] = {};
    if (fits[a.nsplit] == 0) {
      int n_clusters = 0;
      fits[a.nsplit] = cudaOccupancyMaxActiveClusters(&n_clusters, decode_gqa_mma_kernel<D, NWARP, NG, FUSED>, &lc) == cudaSuccess &&
                               n_clusters >= 1 ? 1 : -1;
      if (fits[a.nsplit] < 0) (void)cudaGetLastError();
    }
    if (fits[a.nsplit] < 0) return cudaErrorInvalidClusterSize;
    e = cudaLaunchKernelEx(&lc, decode_gqa_mma_kernel<D, NWARP, NG, FUSED>, a, tk, tv);
    if (e != cudaSuccess) return e;
  } else {
    e = launch_pdl(decode_gqa_mma_kernel<D, NWARP, NG, FUSED>, dim3(a.nsplit, a.Hkv, n_active), dim3(NWARP * 32), smem, st, a, tk, tv);
  }
  count_launch();
  return e;
}

}  // namespace

bool decode_gqa_mma_supported(int dtype, const Shape& s) {
  return dtype == SNAP_BF16 && s.d_qk == s.d_v && (s.d_qk == 64 || s.d_qk == 128 || s.d_qk == 256) && !s.v_aliases_k &&
         s.g >= 1 && s.g <= 2 * GP && umma::encode_tiled_fn() != nullptr;
}

size_t decode_gqa_mma_partial_floats(const Shape& s, int n_rows, int nsplit) {
  return (size_t)n_rows * s.Hq * nsplit * (s.d_v + 2);
}

cudaError_t launch_decode_gqa_mma(const Shape& s, const void* q, const void* k_new, const void* v_new,
                                  const int* slot_ids, int n_active, void* k_cache, void* v_cache,
                                  int* seq_len, const int* valid_topk, void* out, float* partials,
                                  int nsplit, uint32_t* status, cudaStream_t st, int q_len, int q_total, int u0,
                                  const int* block_idx, const int* n_sel, int blocks_cap, int block_tokens) {
  if (n_active == 0) return cudaSuccess;
  if (block_idx && (!n_sel || blocks_cap < 1 || block_tokens < WT || block_tokens % WT || q_len != 1)) return cudaErrorInvalidValue;
  if (q_total < q_len) { q_total = q_len; u0 = 0; }            // the launch's tokens are all the step's tokens
  if (q_len < 1 || q_len * s.g > 2 * GP || (q_len > 1 && (!k_new || q_len > s.Lr)) || u0 < 0 || u0 + q_len > q_total)
    return cudaErrorInvalidValue;
  umma::EncodeTiledFn enc = umma::encode_tiled_fn();
  if (!enc) return cudaErrorNotSupported;
  const int D = s.d_qk;
  // The two tensor maps depend only on the cache buffers and their shape: keep the last few per
  // host thread instead of encoding them on every decode step.
  struct MapEntry { const void* k; const void* v; int Sc, d; long long planes; CUtensorMap tk, tv; };
  constexpr int kMapCache = 8;
  thread_local MapEntry cache[kMapCache] = {};
  thread_local int cache_next = 0;
  const long long planes = (long long)s.max_seqs * s.Hkv;
  const MapEntry* hit = nullptr;
  for (int e = 0; e < kMapCache; ++e)
    if (cache[e].k == k_cache && cache[e].v == v_cache && cache[e].Sc == s.Sc && cache[e].d == D && cache[e].planes == planes &&
        cache[e].k) {
      hit = &cache[e];
      break;
    }
  if (!hit) {
    MapEntry& m = cache[cache_next];
    cache_next = (cache_next + 1) % kMapCache;
    const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)s.Sc, (cuuint64_t)planes};
    const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)s.Sc * D * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)WT, 1}, estr[3] = {1, 1, 1};
    m.k = nullptr;
    if (enc(&m.tk, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, k_cache, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
        enc(&m.tv, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, v_cache, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
    m.k = k_cache; m.v = v_cache; m.Sc = s.Sc; m.d = D; m.planes = planes;
    hit = &m;
  }
  MmaArgs a;
  a.q = static_cast<const __nv_bfloat16*>(q);
  a.k_new = static_cast<const __nv_bfloat16*>(k_new);
  a.v_new = static_cast<const __nv_bfloat16*>(v_new);
  a.slot_ids = slot_ids;
  a.kc = static_cast<char*>(k_cache); a.vc = static_cast<char*>(v_cache);
  a.head_b = (long long)s.Sc * D * 2; a.seq_b = a.head_b * s.Hkv;
  a.Hq = s.Hq; a.Hkv = s.Hkv; a.g = s.g; a.Ls = s.Ls; a.Lr = s.Lr; a.max_seqs = s.max_seqs; a.nsplit = nsplit;
  a.T = q_len; a.QT = q_total; a.u0 = u0;
  a.scale_log2 = s.scale * 1.4426950408889634f;
  a.seq_len = seq_len; a.valid_topk = valid_topk; a.partials = partials; a.status = status;
  a.block_idx = block_idx; a.n_sel = n_sel; a.blocks_cap = blocks_cap; a.tpb = block_idx ? block_tokens / WT : 1;
  cudaError_t e;
  const bool wide = q_len * s.g > GP;                          // 9 to 16 (token, head) columns: two column groups
  // Small batches (the grid is at most about one CTA per SM) whose step is being captured into a CUDA graph: the
  // splits merge inside the kernel, as one cluster per (sequence, KV head) -- 9.6 against 11.0 us per replayed
  // step of one 5124-slot sequence.  Launched eagerly such a step is bound by the host's launch calls, and a
  // cluster launch costs the host more than the merge kernel's plain launch (16.3 against 12.0 us per step), so
  // eager steps keep the two launches.  Option SNAP_OPT_DECODE_GQA_KERNEL = 2: never merge in the kernel, 3: merge
  // in the kernel whenever the shape allows (testing aids).  A device that refuses the cluster shape gets the
  // two launches from then on.
  static bool fused_refused = false;
  bool fused = !wide && q_len == 1 && nsplit >= 2 && nsplit <= 16 && !fused_refused && option(SNAP_OPT_DECODE_GQA_KERNEL) != 2 &&
               (long long)nsplit * s.Hkv * n_active <= 160;
  if (fused && option(SNAP_OPT_DECODE_GQA_KERNEL) != 3) {
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    fused = cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusActive;
  }
  if (fused) {
    a.out = static_cast<__nv_bfloat16*>(out);
    e = D == 128 ? launch_d<128, 4, 1, true>(a, hit->tk, hit->tv, n_active, st)
        : D == 64 ? launch_d<64, 4, 1, true>(a, hit->tk, hit->tv, n_active, st)
                  : launch_d<256, 2, 1, true>(a, hit->tk, hit->tv, n_active, st);
    if (e == cudaSuccess) {
      if (!k_new) return cudaGetLastError();                   // attend only: the lengths stay
      e = launch_pdl(decode_gqa_bump_kernel, dim3((n_active + 127) / 128), dim3(128), 0, st, slot_ids, seq_len, s.max_seqs, n_active, 1);
      count_launch();
      return e != cudaSuccess ? e : cudaGetLastError();
    }
    (void)cudaGetLastError();                                  // e.g. a cluster of this size cannot be scheduled: two launches from now on
    fused_refused = true;
  }
  a.out = nullptr;
  if (D == 128) e = wide ? launch_d<128, 4, 2, false>(a, hit->tk, hit->tv, n_active, st) : launch_d<128, 4, 1, false>(a, hit->tk, hit->tv, n_active, st);
  else if (D == 64) e = wide ? launch_d<64, 4, 2, false>(a, hit->tk, hit->tv, n_active, st) : launch_d<64, 4, 1, false>(a, hit->tk, hit->tv, n_active, st);
  else e = wide ? launch_d<256, 2, 2, false>(a, hit->tk, hit->tv, n_active, st) : launch_d<256, 2, 1, false>(a, hit->tk, hit->tv, n_active, st);
  if (e != cudaSuccess) return e;
  if (D == 128)
    return launch_decode_gqa_merge(partials, out, s.Hq, nsplit, slot_ids, n_active * q_len, q_len, seq_len, s.max_seqs,
                                   k_new != nullptr, st, q_total, u0);
  e = launch_pdl(decode_gqa_mma_merge_kernel, dim3(s.Hq, n_active * q_len), dim3(128), 0, st,
                 static_cast<const float*>(partials), static_cast<__nv_bfloat16*>(out), s.Hq, D, nsplit, slot_ids, seq_len,
                 s.max_seqs, (int)(k_new != nullptr), q_len, q_total, u0);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace snap
