// Causal prefill attention on tcgen05 that also emits the normalisers of Eq. 4 for the
// observation window (Section 3.2.2 leaves the score recomputation as a step to optimise: the
// denominators of the scores are by-products of the prompt's own attention pass, so the first of
// the two passes of the score kernel can be dropped when the prompt's attention ran here).
//
// A CTA computes 128 query rows of one head, or of two heads that share a KV head, against key
// tiles 0 .. its own (128 keys each):
//   S = Q K^T      M = 128 rows, N = 128 keys, both operands K-major in shared memory
//   O += P V       A = P from tensor memory (bf16 pairs written over the tile's own logits),
//                  B = the V tile as loaded (MN-major)
// K and V tiles stream through a ring of four 32 KB stages in the order the MMAs consume them.
//   warp 0      TMA producer
//   warp 1      MMA issuer (whole warp converged, instructions predicated on one lane)
//   warps 2-5 (and 6-9 for the second head)
//               thread = query row: online softmax in the log2 domain with a lazily refreshed
//               reference (O is rescaled in tensor memory only when a logit exceeds it by 8);
//               the arithmetic around the exponentials is packed two-wide, and P is handed to
//               the MMA warp in two halves of 64 keys
// Rows of the last Lo positions also accumulate the same exponentials over the eviction
// candidates [Ls, L - Lr) alone; reference + log2 of that sum is what Eq. 4 divides by.
// Every mbarrier wait is bounded; one that runs out raises SNAP_DEV_WAIT_TIMEOUT.
#include <cstdlib>

#include "snap_internal.cuh"
#include "umma_helpers.cuh"

namespace snap {
namespace {

using namespace umma;

constexpr int D = 128, BM = 128, BN = 128, NSTG = 4;
constexpr int SLAB_B = 128 * 128, TILE_B = 2 * SLAB_B;           // a tile = two 64-dim slabs of 128 rows x 128 B
constexpr uint32_t COL_S = 0, COL_O = 256;

struct PArgs {
  SeqBatch b;
  int Hq, g, Ls, Lr, Lo;
  float scale_log2;
  __nv_bfloat16* out;                          // [tokens][Hq][D]
  float* mu;                                   // NULL or [prompts][Hq][Lo]
  uint32_t* status;
};

// NQ = 1: one head per CTA; tensor memory S0 128 | S1 128 | O 128 columns, S double-buffered
// (the next tile's logits are computed while the softmax warps work on this one).
// NQ = 2: two query heads of one KV head per CTA, each with its own softmax warpgroup, S and O
// (4 x 128 columns: tensor memory is full).  They share every K and V tile, which halves the
// traffic from L2, and while one head's warps work the tensor core serves the other head: a
// head's next S follows its P V (its logits are overwritten by its probabilities).
template <int NQ>
__global__ void __launch_bounds__(64 + 128 * NQ, 1)
prefill_attn_kernel(const PArgs a, const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                    const __grid_constant__ CUtensorMap tmap_v) {
  const int seq = blockIdx.z, head0 = blockIdx.y * NQ;
  const int L = a.b.len[seq];
  const int n_qt = (L + BM - 1) / BM;
  if ((int)blockIdx.x >= n_qt) return;                         // the grid is sized for the longest prompt
  const int qt = n_qt - 1 - (int)blockIdx.x;                   // longest rows first
  const int q0 = qt * BM, nt = qt + 1;
  const int tok0 = a.b.tok_off[seq], kvh = head0 / a.g;

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* Qs = smem;                                    // [NQ heads][2 slabs][128 rows][128 B]
  unsigned char* Rs = Qs + NQ * TILE_B;                        // [NSTG][32 KB] ring
  uint64_t* bars = reinterpret_cast<uint64_t*>(Rs + NSTG * TILE_B);
  // full[NSTG] empty[NSTG] s_full[2] p_ready[2][2 halves of the keys] pv_done[2] q_full
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * NSTG + 9);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8 * s; };
  auto empty_bar = [&](int s) { return bar0 + 8 * (NSTG + s); };
  auto sfull_bar = [&](int b) { return bar0 + 8 * (2 * NSTG + b); };
  auto pready_bar = [&](int b, int half) { return bar0 + 8 * (2 * NSTG + 2 + 2 * b + half); };
  auto pvdone_bar = [&](int b) { return bar0 + 8 * (2 * NSTG + 6 + b); };
  const uint32_t qfull_bar = bar0 + 8 * (2 * NSTG + 8);
  // S / P buffer, its barriers and their phase for tile `it` of head x:
  //   NQ = 1: two buffers used alternately by the one head; NQ = 2: one buffer per head
  auto buf_of = [&](int x, int it) { return NQ == 1 ? (it & 1) : x; };
  auto phase_of = [&](int it) { return NQ == 1 ? ((unsigned)(it / 2) & 1u) : ((unsigned)it & 1u); };

  if (tid == 0) {
    *abort_flag = 0;
    for (int s = 0; s < NSTG; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(sfull_bar(b), 1); mbar_init(pready_bar(b, 0), 4); mbar_init(pready_bar(b, 1), 4); mbar_init(pvdone_bar(b), 1);
    }
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

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      mbar_expect_tx(qfull_bar, (unsigned)(NQ * TILE_B));
      for (int x = 0; x < NQ; ++x)
        for (int h = 0; h < 2; ++h)
          tma_load_3d(smem_u32(Qs) + x * TILE_B + h * SLAB_B, &tmap_q, h * 64, head0 + x, tok0 + q0, qfull_bar);
      int q = 0;                                               // stages issued so far
      bool ok = true;
      auto load_tile = [&](const CUtensorMap* map, int it) {
        const int s = q % NSTG;
        if (!mbar_wait(empty_bar(s), ((unsigned)(q / NSTG) & 1u) ^ 1u, abort_flag)) { *abort_flag = 1; ok = false; return; }
        mbar_expect_tx(full_bar(s), (unsigned)TILE_B);
        for (int h = 0; h < 2; ++h)
          tma_load_3d(smem_u32(Rs) + s * TILE_B + h * SLAB_B, map, h * 64, kvh, tok0 + it * BN, full_bar(s));
        ++q;
      };
      // in the order the MMA warp consumes: NQ = 1: K(0), K(1), V(0), K(2), V(1), ...
      //                                     NQ = 2: K(0), V(0), K(1), V(1), ...
      load_tile(&tmap_k, 0);
      for (int it = 0; it < nt && ok; ++it) {
        if (NQ == 1) {
          if (it + 1 < nt) load_tile(&tmap_k, it + 1);
          if (ok) load_tile(&tmap_v, it);
        } else {
          load_tile(&tmap_v, it);
          if (ok && it + 1 < nt) load_tile(&tmap_k, it + 1);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    const uint32_t leader = lane == 0;
    const uint32_t idesc_s = idesc_f16(BM, BN, false), idesc_pv = idesc_f16(BM, D, true);
    const uint64_t qd0 = smem_desc(smem_u32(Qs));
    int q = 0;                                                 // stages consumed so far
    bool ok = wait_warp(qfull_bar, 0u, abort_flag);
    fence_after();
    auto wait_stage = [&]() -> bool {
      const bool r = wait_warp(full_bar(q % NSTG), (unsigned)(q / NSTG) & 1u, abort_flag);
      fence_after();
      return r;
    };
    auto issue_s = [&](int x, int it, int s) {                // S of head x = Q_x K(it)^T, K in stage s
      const uint32_t sd = tmem_base + COL_S + buf_of(x, it) * BN;
      const uint64_t kd0 = smem_desc(smem_u32(Rs) + s * TILE_B), qdx = qd0 + (uint64_t)((x * TILE_B) >> 4);
      // one instruction group per 64-dim slab: this warp's instruction chain per MMA is what the tensor pipe waits for
#pragma unroll
      for (int h = 0; h < 2; ++h)
        mma_ss_slab4_pred(sd, qdx + (uint64_t)((h * SLAB_B) >> 4), kd0 + (uint64_t)((h * SLAB_B) >> 4), idesc_s, h != 0, leader);
      commit_pred(sfull_bar(buf_of(x, it)), leader);
    };
    auto issue_pv = [&](int x, int it, int s) -> bool {       // O_x += P_x(it) V(it), V in stage s
      const uint32_t vst = smem_u32(Rs) + s * TILE_B;
      const uint32_t pa = tmem_base + COL_S + buf_of(x, it) * BN;   // P lies over the first 64 columns of its S
#pragma unroll
      for (int half = 0; half < 2; ++half) {                  // the first 64 keys go while the rest are exponentiated
        if (!wait_warp(pready_bar(buf_of(x, it), half), phase_of(it), abort_flag)) return false;
        fence_after();
        // four instructions of 16 keys each, one group
        mma_ts_4_pred(tmem_base + COL_O + x * D, pa + 32 * half, smem_desc_mn(vst + half * 64 * 128, SLAB_B), (16 * 128) >> 4,
                      idesc_pv, (it | half) != 0, leader);
      }
      commit_pred(pvdone_bar(buf_of(x, it)), leader);
      return true;
    };
    auto clear_ragged_v = [&](int it, int s) {
      const int tile_nrows = L - it * BN;
      if (tile_nrows < BN) {
        // rows past the prompt's end hold another prompt's tokens or nothing at all, and a zero
        // probability does not silence a NaN in V: clear them before the tensor core reads
        for (int e = lane; e < (BN - tile_nrows) * 16; e += 32) {
          const int r = tile_nrows + e / 16, j = (e / 8) % 2, ch = e % 8;
          *reinterpret_cast<uint4*>(Rs + s * TILE_B + j * SLAB_B + r * 128 + ch * 16) = make_uint4(0, 0, 0, 0);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
      }
    };
    if (ok) ok = wait_stage();
    if (ok) {
      for (int x = 0; x < NQ; ++x) issue_s(x, 0, q % NSTG);
      commit_pred(empty_bar(q % NSTG), leader);
      ++q;
    }
    for (int it = 0; it < nt && ok; ++it) {
      if (NQ == 1) {
        if (it + 1 < nt) {
          ok = wait_stage();
          if (!ok) break;
          issue_s(0, it + 1, q % NSTG);
          commit_pred(empty_bar(q % NSTG), leader);
          ++q;
        }
        ok = wait_stage();
        if (!ok) break;
        clear_ragged_v(it, q % NSTG);
        ok = issue_pv(0, it, q % NSTG);
        if (!ok) break;
        commit_pred(empty_bar(q % NSTG), leader);
        ++q;
      } else {
        // a head's next logits go where its probabilities are, so they follow its P V; the other
        // head's instructions fill the time its softmax warps need
        ok = wait_stage();
        if (!ok) break;
        const int sv = q % NSTG;
        ++q;
        clear_ragged_v(it, sv);
        const bool more = it + 1 < nt;
        int sk = 0;
        ok = issue_pv(0, it, sv);
        if (!ok) break;
        if (more) {
          ok = wait_stage();
          if (!ok) break;
          sk = q % NSTG;
          ++q;
          issue_s(0, it + 1, sk);
        }
        ok = issue_pv(1, it, sv);
        if (!ok) break;
        commit_pred(empty_bar(sv), leader);
        if (more) {
          issue_s(1, it + 1, sk);
          commit_pred(empty_bar(sk), leader);
        }
      }
    }
    if (!ok && lane == 0) *abort_flag = 1;
  } else {
    // ---------------- softmax warps: thread = query row, one warpgroup per head ----------------
    const int x = (warp - 2) >> 2, head = head0 + x;
    const int lrow = 32 * (warp & 3) + lane;                   // TMEM lane
    const uint32_t lane_addr = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16);
    const uint32_t o_addr = lane_addr + COL_O + x * D;
    const int row = q0 + lrow;                                 // position within the prompt
    // does this warp hold rows of the observation window?  (warp-uniform)
    const int wrow0 = q0 + 32 * (warp & 3);
    const bool warp_window = a.mu != nullptr && wrow0 + 31 >= L - a.Lo && wrow0 < L;
    const int cand_lo = a.Ls, cand_n = L - a.Lr - a.Ls;        // candidates [cand_lo, cand_lo + cand_n)
    const float sc = a.scale_log2;                             // > 0: the largest raw logit is the largest scaled one
    float m_ref = -INFINITY, l_sum = 0.f, l_cand = 0.f;
    bool ok = true;
    for (int it = 0; it < nt; ++it) {
      const int b = buf_of(x, it);
      if (!wait_warp(sfull_bar(b), phase_of(it), abort_flag)) { ok = false; break; }
      fence_after();
      const uint32_t s_addr = lane_addr + COL_S + b * BN;
      float v[BN];                                             // raw logits
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
      if (it == nt - 1) {
        // the tile on the diagonal: key j of the tile is visible to row lrow iff j <= lrow
#pragma unroll
        for (int j = 0; j < BN; ++j) v[j] = j <= lrow ? v[j] : -INFINITY;
      }
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int j = 0; j < BN; j += 4) {
        mx0 = fmaxf(mx0, fmaxf(v[j], v[j + 1]));
        mx1 = fmaxf(mx1, fmaxf(v[j + 2], v[j + 3]));
      }
      float mx = fmaxf(mx0, mx1);
      mx *= sc;
      // Lazy reference: refreshed (and O rescaled) only when some row of the warp sees a logit 8
      // above its reference; the tensor-memory accesses are warp-collective, so the warp votes.
      if (__any_sync(0xffffffffu, mx > m_ref + 8.f)) {
        const float m_new = fmaxf(m_ref, mx);
        const float alpha = m_ref == -INFINITY ? 0.f : exp2f(m_ref - m_new);
        if (it > 0) {
          if (!wait_warp(pvdone_bar(buf_of(x, it - 1)), phase_of(it - 1), abort_flag)) { ok = false; break; }
          fence_after();
#pragma unroll 1
          for (int c = 0; c < D / 16; ++c) {
            uint32_t o[16];
            tmem_ld16_issue(o_addr + 16 * c, o);
            tmem_ld16_wait(o);
#pragma unroll
            for (int e = 0; e < 16; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st16(o_addr + 16 * c, o);
          }
          tmem_st_wait();
        }
        l_sum *= alpha;
        l_cand *= alpha;
        m_ref = m_new;
      }
      const float nmr = m_ref == -INFINITY ? 0.f : -m_ref;
      float ls0 = 0.f, ls1 = 0.f;
      // this tile's overlap with the candidate range, as tile columns [clo, clo + cn)
      const int clo = cand_lo - it * BN;
      const unsigned cn = warp_window && cand_n > 0 ? (unsigned)cand_n : 0u;
      // the logits of this tile are all in registers, so the probabilities may overwrite them
      u64 ls2 = pack2(0.f, 0.f);
      const u64 sc2 = pack2(sc, sc), nmr2 = pack2(nmr, nmr);
#pragma unroll
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t pk[16];
        if (!warp_window) {
          // two-wide multiply-adds and sums: the arithmetic around the exponentials takes half the issue slots
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const u64 x2 = fma2(pack2(v[32 * c + 2 * j], v[32 * c + 2 * j + 1]), sc2, nmr2);
            const float p0 = fast_exp2(lo2(x2)), p1 = fast_exp2(hi2(x2));
            ls2 = add2(ls2, pack2(p0, p1));
            pk[j] = pack_bf16(p0, p1);
          }
        } else {
          // rows of the observation window also sum over the candidate columns alone
          float pc = 0.f;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float p0 = fast_exp2(fmaf(v[32 * c + 2 * j], sc, nmr)), p1 = fast_exp2(fmaf(v[32 * c + 2 * j + 1], sc, nmr));
            ls0 += p0;
            ls1 += p1;
            pc += (unsigned)(32 * c + 2 * j - clo) < cn ? p0 : 0.f;
            pc += (unsigned)(32 * c + 2 * j + 1 - clo) < cn ? p1 : 0.f;
            pk[j] = pack_bf16(p0, p1);
          }
          l_cand += pc;
        }
        tmem_st16(s_addr + 16 * c, pk);
        if (c & 1) {                                           // a half of the keys is complete
          tmem_st_wait();
          fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(pready_bar(b, c >> 1));
        }
      }
      ls0 += lo2(ls2);
      ls1 += hi2(ls2);
      l_sum += ls0 + ls1;
    }
    if (!ok) *abort_flag = 1;
    // ---------------- normalise and store ----------------
    if (ok) ok = wait_warp(pvdone_bar(buf_of(x, nt - 1)), phase_of(nt - 1), abort_flag);
    if (!ok) *abort_flag = 1;
    fence_after();
    if (__all_sync(0xffffffffu, ok)) {
      const float inv = 1.f / l_sum;
      __nv_bfloat16* orow = a.out + ((long long)(tok0 + row) * a.Hq + head) * D;
#pragma unroll 1
      for (int c = 0; c < D / 16; ++c) {
        uint32_t o[16];
        tmem_ld16_issue(o_addr + 16 * c, o);
        tmem_ld16_wait(o);
        if (row < L) {
          uint4 w0, w1;
          w0.x = pack_bf16(__uint_as_float(o[0]) * inv, __uint_as_float(o[1]) * inv);
          w0.y = pack_bf16(__uint_as_float(o[2]) * inv, __uint_as_float(o[3]) * inv);
          w0.z = pack_bf16(__uint_as_float(o[4]) * inv, __uint_as_float(o[5]) * inv);
          w0.w = pack_bf16(__uint_as_float(o[6]) * inv, __uint_as_float(o[7]) * inv);
          w1.x = pack_bf16(__uint_as_float(o[8]) * inv, __uint_as_float(o[9]) * inv);
          w1.y = pack_bf16(__uint_as_float(o[10]) * inv, __uint_as_float(o[11]) * inv);
          w1.z = pack_bf16(__uint_as_float(o[12]) * inv, __uint_as_float(o[13]) * inv);
          w1.w = pack_bf16(__uint_as_float(o[14]) * inv, __uint_as_float(o[15]) * inv);
          reinterpret_cast<uint4*>(orow + 16 * c)[0] = w0;
          reinterpret_cast<uint4*>(orow + 16 * c)[1] = w1;
        }
      }
      const int w = row - (L - a.Lo);
      if (warp_window && row < L && w >= 0)
        a.mu[((long long)(a.b.first_seq + seq) * a.Hq + head) * a.Lo + w] = l_cand > 0.f ? m_ref + log2f(l_cand) : -INFINITY;
    }
  }

  fence_before();
  __syncthreads();
  fence_after();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  if (tid == 0 && *abort_flag && a.status) atomicOr(a.status, SNAP_DEV_WAIT_TIMEOUT);
}

size_t prefill_smem_bytes(int nq) { return (size_t)nq * TILE_B + NSTG * TILE_B + (2 * NSTG + 9) * 8 + 16 + 1024; }

}  // namespace

bool prefill_attn_supported(int dtype, const Shape& s) {
  return dtype == SNAP_BF16 && !s.v_aliases_k && s.d_qk == D && s.d_v == D && umma::encode_tiled_fn() != nullptr;
}

cudaError_t launch_prefill_attn(const Shape& s, const SeqBatch& b, const void* q, const KVSource& src, void* out,
                                float* mu, uint32_t* status, cudaStream_t st) {
  long long tokens = 0;
  int max_len = 0;
  for (int i = 0; i < b.n; ++i) {
    tokens = tokens > (long long)b.tok_off[i] + b.len[i] ? tokens : (long long)b.tok_off[i] + b.len[i];
    max_len = max_len > b.len[i] ? max_len : b.len[i];
  }
  if (b.n == 0 || max_len == 0) return cudaSuccess;
  umma::EncodeTiledFn enc = umma::encode_tiled_fn();
  if (!enc) return cudaErrorNotSupported;
  CUtensorMap tq, tk, tv;
  const cuuint32_t estr[3] = {1, 1, 1};
  const cuuint32_t box[3] = {64, 1, (cuuint32_t)BM};
  auto encode = [&](CUtensorMap* m, const void* base, int heads, long long head_stride, long long tok_stride) {
    const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)heads, (cuuint64_t)tokens};
    const cuuint64_t strides[2] = {(cuuint64_t)(head_stride >= D ? head_stride : D) * 2, (cuuint64_t)tok_stride * 2};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
  };
  if (!encode(&tq, q, s.Hq, D, (long long)s.Hq * D) || !encode(&tk, src.k, s.Hkv, src.k_head_stride, src.k_tok_stride) ||
      !encode(&tv, src.v, s.Hkv, src.v_head_stride, src.v_tok_stride))
    return cudaErrorInvalidValue;
  PArgs a;
  a.b = b;
  a.Hq = s.Hq; a.g = s.g; a.Ls = s.Ls; a.Lr = s.Lr; a.Lo = s.Lo;
  a.scale_log2 = s.scale * 1.4426950408889634f;
  a.out = static_cast<__nv_bfloat16*>(out);
  a.mu = mu;
  a.status = status;
  // pairs of heads that share a KV head when the group allows (option SNAP_OPT_PREFILL_SINGLE_HEADS forces single heads)
  const int nq = s.g % 2 == 0 && option(SNAP_OPT_PREFILL_SINGLE_HEADS) != 1 ? 2 : 1;
  const size_t smem = prefill_smem_bytes(nq);
  static SmemLimit limit1 = {}, limit2 = {};
  const dim3 grid((max_len + BM - 1) / BM, s.Hq / nq, b.n);
  if (nq == 2) {
    if (cudaError_t e = ensure_dyn_smem(prefill_attn_kernel<2>, smem, limit2)) return e;
    prefill_attn_kernel<2><<<grid, 64 + 128 * 2, smem, st>>>(a, tq, tk, tv);
  } else {
    if (cudaError_t e = ensure_dyn_smem(prefill_attn_kernel<1>, smem, limit1)) return e;
    prefill_attn_kernel<1><<<grid, 64 + 128, smem, st>>>(a, tq, tk, tv);
  }
  count_launch();
  return cudaGetLastError();
}

}  // namespace snap
