// Observation-window scores on the 5th-generation tensor cores (Eq. 4 -> Eq. 1 with the GQA
// group sum): tcgen05.mma with accumulators in tensor memory, operands staged by TMA.
// Covers bf16 layers with 128-wide heads and 128 or 256 window rows per KV head (g * Lo).
//
// One CTA per SM, warp specialised, persistent over a run of 128-candidate tiles:
//   warp 0   TMA producer: the query block once, then key tiles into a ring of four stages (three
//            in pass 2) (cp.async.bulk.tensor, 128-byte swizzle, two 64-element K halves per tile)
//   warp 1   MMA issuer: one elected thread issues tcgen05.mma (M128, K16 steps) from shared
//            memory descriptors into one of two TMEM accumulator buffers and commits to mbarriers
//   warps 2-9  epilogue: read the accumulators with tcgen05.ld (thread = TMEM lane) while the
//            next tile's MMAs run into the other buffer
//
// Pass 1 puts the query rows on M (two 128-row blocks share each key tile; N = 128 candidates),
// so a thread owns one query row and keeps that row's running (reference max, sum of exp2) with
// no cross-thread traffic.  Pass 2 puts the candidates on M (N = all query rows), so a thread
// owns one candidate, and carries the normalisers in the contraction: one more 16-wide step adds
// -mu_i / scale (mu_i = m_i + log2 l_i, split into bf16 pieces against ones) to column i, so the
// epilogue is a plain sum of exp2(scale * acc).  The two epilogue groups each sum half of the
// columns, group 1 hands its partial to group 0 through shared memory, and group 0 stores C[j].
// The reference max of pass 1 is refreshed lazily (only when a tile's partial sum shows a logit
// far above it).  Statistics are in the log2 domain.  Every mbarrier wait is bounded; a wait
// that runs out raises SNAP_DEV_WAIT_TIMEOUT and the CTA drains and frees its tensor memory.
#include <cuda.h>

#include <cstdlib>

#include "snap_internal.cuh"
#include "umma_helpers.cuh"

namespace snap {
namespace {

using namespace umma;

constexpr int D = 128, TN = 128;
constexpr int kStagesPass1 = 4, kStagesPass2 = 3;          // pass 2 gives one stage up for its extra operand slabs
constexpr int HALF_B = TN * 128;             // one K half of a 128-row tile: 128 rows x 128 bytes
constexpr int STAGE_B = 2 * HALF_B;          // 32 KB
constexpr int NTHREADS = 320;                // 10 warps

struct UmmaArgs {
  int Hq, Hkv, g, Lo, Ls, Lr, R;
  float scale_log2;
  SeqBatch b;
  ScoreBuffers buf;
  uint32_t* status;
};

// acc (two pairs, alternated) += exp2(r[i] * scale + off) over 2 n raw logits, off the same for all
template <int N2>
__device__ __forceinline__ void exp_sum_const(const uint32_t* r, u64 sc2, u64 off2, u64 (&acc)[2]) {
#pragma unroll
  for (int i = 0; i < N2; ++i) {
    const u64 x = fma2(pack2(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1])), sc2, off2);
    acc[i & 1] = add2(acc[i & 1], pack2(fast_exp2(lo2(x)), fast_exp2(hi2(x))));
  }
}
template <int PASS>
__global__ void __launch_bounds__(NTHREADS, 1)
score_umma_kernel(const UmmaArgs a, const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int R = a.R, MB = R / 128;
  constexpr int NS = PASS == 1 ? kStagesPass1 : kStagesPass2;
  unsigned char* Qs = smem;                                   // [2 halves][R][128 B]
  unsigned char* Ks = Qs + R * 256;                           // [NS][2 halves][128][128 B]
  // pass 2: one more 16-wide step of the contraction, whose operands are constants of the launch
  unsigned char* tail = Ks + NS * STAGE_B;
  unsigned char* Qx = tail;                                   // [256][128 B]  row i: -mu_i / scale as four bf16 pieces
  unsigned char* Kx = Qx + 256 * 128;                         // [128][128 B]  ones against those pieces
  float2* stats_s = reinterpret_cast<float2*>(PASS == 2 ? Kx + HALF_B : tail);   // [R] floats: mu_i (pass 2)
  float2* xch = stats_s + 256;                                // [128] pass-1 exchange between epilogue groups
  uint64_t* bars = reinterpret_cast<uint64_t*>(xch + 128);    // full[NS] empty[NS] tfull[2] tempty[2] qfull xfull[2] xempty[2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * NS + 9);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int z = blockIdx.y, si = z / a.Hkv, kvh = z % a.Hkv;
  const int seq = a.b.seq_of_score[si];
  const int Le = a.b.len[seq] - a.Ls - a.Lr;
  const int ntiles = (Le + TN - 1) / TN;
  // equal chunks of candidate tiles for every prompt of the launch: a shorter prompt uses fewer of the splits
  const int t0 = min(ntiles, (int)blockIdx.x * a.buf.chunk_tiles);
  const int t1 = min(ntiles, t0 + a.buf.chunk_tiles);
  const int nt = t1 - t0;
  // Both epilogue groups work on every tile -- pass 1 with two row blocks (one block each) and pass 2
  // (half of the accumulator columns each) -- so that a tile's buffer is free again after half the
  // time and the next MMA never waits for it; pass 1 with one row block alternates tiles instead.
  const bool both = PASS == 2 || MB == 2;

  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8 * s; };
  auto empty_bar = [&](int s) { return bar0 + 8 * (NS + s); };
  auto tfull_bar = [&](int b) { return bar0 + 8 * (2 * NS + b); };
  auto tempty_bar = [&](int b) { return bar0 + 8 * (2 * NS + 2 + b); };
  const uint32_t qfull_bar = bar0 + 8 * (2 * NS + 4);
  auto xfull_bar = [&](int b) { return bar0 + 8 * (2 * NS + 5 + b); };    // pass 2: group 1's partial sums are in xch
  auto xempty_bar = [&](int b) { return bar0 + 8 * (2 * NS + 7 + b); };   //         ... and have been taken

  if (tid == 0) {
    *abort_flag = 0;
    for (int s = 0; s < NS; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), both ? 8 : 4); }
    mbar_init(qfull_bar, 1);
    for (int b = 0; b < 2; ++b) { mbar_init(xfull_bar(b), 4); mbar_init(xempty_bar(b), 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  pdl_wait();                                                 // everything above overlaps the previous kernel's tail
  float* mu_s = reinterpret_cast<float*>(stats_s);            // pass 2: m_i + log2(l_i) per query row
  if (PASS == 2) {
    // the g * Lo rows of a KV head are consecutive in [prompt][Hq][Lo] order
    const float* ext = a.buf.ext_mu ? a.buf.ext_mu + ((long long)(a.b.first_seq + seq) * a.Hq + kvh * a.g) * a.Lo : nullptr;
    for (int i = tid; i < R; i += NTHREADS) {
      if (ext) {
        mu_s[i] = ext[i];
      } else {
        const float2 st = a.buf.stats[(long long)z * R + i];
        mu_s[i] = st.x - log2f(st.y);
      }
    }
    __syncthreads();
    // Fold the normalisers into the contraction: one more 16-wide step whose B rows hold
    // -mu_i / scale split into four bf16 pieces (their sum is the fp32 value exactly) and whose A rows hold
    // ones, so that the accumulator is q_i . k_j - mu_i / scale and the epilogue is exp2(scale * acc)
    // with no per-row constant.  Rows of 128 bytes, 128-byte swizzle, only chunks 0 and 1 are read.
    const float inv_scale = 1.f / a.scale_log2;
    for (int i = tid; i < 256 + 128; i += NTHREADS) {
      uint4 c0 = make_uint4(0u, 0u, 0u, 0u);
      unsigned char* rowp;
      if (i < 256) {
        rowp = Qx + i * 128;
        if (i < R) {
          const float c = -mu_s[i] * inv_scale;
          const __nv_bfloat16 hi = __float2bfloat16_rn(c);
          const float r1 = c - __bfloat162float(hi);
          const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
          const float r2 = r1 - __bfloat162float(mid);
          const __nv_bfloat16 lo = __float2bfloat16_rn(r2);
          const __nv_bfloat16 lo2 = __float2bfloat16_rn(r2 - __bfloat162float(lo));   // zero unless c needs all 24 bits
          c0.x = (uint32_t)__bfloat16_as_ushort(hi) | ((uint32_t)__bfloat16_as_ushort(mid) << 16);
          c0.y = (uint32_t)__bfloat16_as_ushort(lo) | ((uint32_t)__bfloat16_as_ushort(lo2) << 16);
        }
      } else {
        rowp = Kx + (i - 256) * 128;
        c0.x = 0x3f803f80u;                                    // bf16 1.0, 1.0
        c0.y = 0x3f803f80u;                                    // bf16 1.0, 1.0
      }
      const int sw = (i < 256 ? i : i - 256) & 7;
      *reinterpret_cast<uint4*>(rowp + ((0 ^ sw) << 4)) = c0;
      *reinterpret_cast<uint4*>(rowp + ((1 ^ sw) << 4)) = make_uint4(0u, 0u, 0u, 0u);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {                                            // tensor memory: 512 columns (2 x 256)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  // epilogue threads: group, accumulator row, and (pass 1) the running statistics of that row
  const int eg = warp >= 2 ? (warp - 2) >> 2 : 0;
  const int lrow = 32 * (warp & 3) + lane;
  float m_ref = -INFINITY, l_sum = 0.f;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0 && nt > 0) {
      const int row0 = ((a.b.first_seq + seq) * a.Hq + kvh * a.g) * a.Lo;
      mbar_expect_tx(qfull_bar, (unsigned)R * 256u);
      for (int h = 0; h < 2; ++h)
        for (int mb = 0; mb < MB; ++mb)
          tma_load_2d(smem_u32(Qs) + h * (R * 128) + mb * HALF_B, &tmap_q, h * 64, row0 + 128 * mb, qfull_bar);
      const int tok0 = a.b.tok_off[seq] + a.Ls;
      for (int it = 0; it < nt; ++it) {
        const int s = it % NS;
        if (!mbar_wait(empty_bar(s), ((unsigned)(it / NS) & 1u) ^ 1u, abort_flag)) { *abort_flag = 1; break; }
        mbar_expect_tx(full_bar(s), (unsigned)STAGE_B);
        const uint32_t dst = smem_u32(Ks) + s * STAGE_B;
        tma_load_3d(dst, &tmap_k, 0, kvh, tok0 + (t0 + it) * TN, full_bar(s));
        tma_load_3d(dst + HALF_B, &tmap_k, 64, kvh, tok0 + (t0 + it) * TN, full_bar(s));
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0 && nt > 0) {
      const uint32_t idesc = PASS == 1 ? idesc_bf16(128, 128) : idesc_bf16(128, R);
      bool ok = mbar_wait(qfull_bar, 0u, abort_flag);
      for (int it = 0; it < nt && ok; ++it) {
        const int s = it % NS, b = it & 1;
        ok = mbar_wait(full_bar(s), (unsigned)(it / NS) & 1u, abort_flag) &&
             mbar_wait(tempty_bar(b), ((unsigned)(it / 2) & 1u) ^ 1u, abort_flag);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t kst = smem_u32(Ks) + s * STAGE_B, qst = smem_u32(Qs);
        // one instruction group per 64-dim slab (four 16-wide steps)
        if (PASS == 1) {
          for (int mb = 0; mb < MB; ++mb)
#pragma unroll
            for (int h = 0; h < D / 64; ++h)
              mma_slab4<false>(tmem_base + b * 256 + mb * 128, smem_desc(qst + h * (R * 128) + mb * HALF_B),
                               smem_desc(kst + h * HALF_B), idesc, h > 0);
        } else {
#pragma unroll
          for (int h = 0; h < D / 64; ++h)
            mma_slab4<false>(tmem_base + b * 256, smem_desc(kst + h * HALF_B), smem_desc(qst + h * (R * 128)), idesc, h > 0);
          mma_bf16(tmem_base + b * 256, smem_desc(smem_u32(Kx)), smem_desc(smem_u32(Qx)), idesc, 1);   // - mu_i / scale
        }
        mma_commit(empty_bar(s));        // the stage may be refilled once these MMAs have read it
        mma_commit(tfull_bar(b));        // the accumulator buffer is complete
      }
      if (!ok) *abort_flag = 1;
    }
  } else {
    // ---------------- epilogue warps ----------------
    // a warp may read the TMEM lane quarter (warp id mod 4); thread = accumulator row lrow
    const uint32_t lane_addr = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16);
    const int mb = both ? eg : 0;
    bool ok = true;
    for (int it = both ? 0 : eg; it < nt; it += both ? 1 : 2) {
      const int b = it & 1;
      const bool landed = mbar_wait(tfull_bar(b), (unsigned)(it / 2) & 1u, abort_flag);
      if (!landed) {
        *abort_flag = 1;
        ok = false;
        break;
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int cand0 = (t0 + it) * TN;
      float part = 0.f;                                        // pass 2: this group's half of the candidate's sum
      if (PASS == 1) {
        const uint32_t col0 = lane_addr + b * 256 + mb * 128;
        const bool full_tile = cand0 + TN <= Le;
        float sum = 0.f;
        float v[32];
        if (full_tile) {
          // software pipeline: the next 32 columns are in flight while these are exponentiated;
          // four partial sums break the dependency chain of the additions
          uint32_t ra[32], rb[32];
          u64 acc[2] = {pack2(0.f, 0.f), pack2(0.f, 0.f)};
          const u64 sc2 = pack2(a.scale_log2, a.scale_log2), nm2 = pack2(-m_ref, -m_ref);
          tmem_ld32_issue(col0, ra);
          tmem_ld_wait(ra);
          tmem_ld32_issue(col0 + 32, rb);
          exp_sum_const<16>(ra, sc2, nm2, acc);
          tmem_ld_wait(rb);
          tmem_ld32_issue(col0 + 64, ra);
          exp_sum_const<16>(rb, sc2, nm2, acc);
          tmem_ld_wait(ra);
          tmem_ld32_issue(col0 + 96, rb);
          exp_sum_const<16>(ra, sc2, nm2, acc);
          tmem_ld_wait(rb);
          exp_sum_const<16>(rb, sc2, nm2, acc);
          sum = (lo2(acc[0]) + hi2(acc[0])) + (lo2(acc[1]) + hi2(acc[1]));
        } else {
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            tmem_ld32(col0 + 32 * c, v);
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const float ex = fast_exp2(fmaf(v[i], a.scale_log2, -m_ref));
              sum += (cand0 + 32 * c + i < Le) ? ex : 0.f;
            }
          }
        }
        // A logit far above the reference (or the first tile): refresh the reference.  The TMEM
        // loads below are warp-collective, so the whole warp takes the branch if any row needs it.
        if (__any_sync(0xffffffffu, !(sum < 65536.f))) {
          float vmax = -INFINITY;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            tmem_ld32(col0 + 32 * c, v);
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (full_tile || cand0 + 32 * c + i < Le) vmax = fmaxf(vmax, v[i] * a.scale_log2);
          }
          const float mn = fmaxf(m_ref, vmax);
          sum = 0.f;
          if (mn != -INFINITY) {
            l_sum *= m_ref == -INFINITY ? 0.f : exp2f(m_ref - mn);
            m_ref = mn;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              tmem_ld32(col0 + 32 * c, v);
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (full_tile || cand0 + 32 * c + i < Le) sum += fast_exp2(fmaf(v[i], a.scale_log2, -mn));
            }
          }
        }
        l_sum += sum;
      } else {
        // thread = candidate: the accumulator row already holds q_i . k_j - mu_i / scale for every
        // query row i of the KV head, so the Eq. 1 score is the plain sum of exp2(scale * acc) over the
        // R columns -- no constants.  This group sums its half of the columns; group 1 hands its
        // partial to group 0 through shared memory (below, after the buffer has been released).
        const uint32_t col0 = lane_addr + b * 256 + eg * (R / 2);
        uint32_t ra[32], rb[32];
        u64 acc[2] = {pack2(0.f, 0.f), pack2(0.f, 0.f)};
        const u64 sc2 = pack2(a.scale_log2, a.scale_log2), zero2 = pack2(0.f, 0.f);
        const int nch = R / 64;                                // 32-column chunks of this half: 2 or 4
        tmem_ld32_issue(col0, ra);
#pragma unroll
        for (int c = 0; c < 4; c += 2) {
          if (c < nch) {
            tmem_ld_wait(ra);
            tmem_ld32_issue(col0 + 32 * (c + 1), rb);
            exp_sum_const<16>(ra, sc2, zero2, acc);
            tmem_ld_wait(rb);
            if (c + 2 < nch) tmem_ld32_issue(col0 + 32 * (c + 2), ra);
            exp_sum_const<16>(rb, sc2, zero2, acc);
          }
        }
        part = (lo2(acc[0]) + hi2(acc[0])) + (lo2(acc[1]) + hi2(acc[1]));
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(b));
      if (PASS == 2) {
        // the two halves of a candidate's sum meet in shared memory (one slot per tile parity)
        float* xs = reinterpret_cast<float*>(xch) + b * 128;
        const unsigned ph = (unsigned)(it / 2) & 1u;
        if (eg == 1) {
          if (!mbar_wait(xempty_bar(b), ph ^ 1u, abort_flag)) { *abort_flag = 1; ok = false; break; }
          xs[lrow] = part;
          __syncwarp();
          if (lane == 0) mbar_arrive(xfull_bar(b));
        } else {
          if (!mbar_wait(xfull_bar(b), ph, abort_flag)) { *abort_flag = 1; ok = false; break; }
          if (cand0 + lrow < Le) a.buf.C[(long long)z * a.buf.c_stride + cand0 + lrow] = part + xs[lrow];
          __syncwarp();
          if (lane == 0) mbar_arrive(xempty_bar(b));
        }
      }
      if (!ok) break;
    }
    if (!ok) *abort_flag = 1;
    if (PASS == 1) {
      if (both)
        a.buf.part_stats[((long long)z * a.buf.nsplit + blockIdx.x) * R + 128 * mb + lrow] = make_float2(m_ref, l_sum);
      else if (eg == 1)
        xch[lrow] = make_float2(m_ref, l_sum);                // merged by group 0 after the barrier below
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  if (PASS == 1 && !both && warp >= 2 && eg == 0) {          // one row block: the two groups took alternate tiles
    const float2 o = xch[lrow];
    merge_ml(m_ref, l_sum, o.x, o.y);
    a.buf.part_stats[((long long)z * a.buf.nsplit + blockIdx.x) * R + lrow] = make_float2(m_ref, l_sum);
  }
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
  if (tid == 0 && *abort_flag && a.status) atomicOr(a.status, SNAP_DEV_WAIT_TIMEOUT);
}

constexpr size_t smem_bytes(int pass) {
  return 256 * 256 + (pass == 1 ? kStagesPass1 * STAGE_B : kStagesPass2 * STAGE_B + 256 * 128 + HALF_B) +
         256 * sizeof(float2) + 128 * sizeof(float2) + (2 * kStagesPass1 + 9) * 8 + 16 + 1024;
}

}  // namespace

bool score_umma_supported(int dtype, const Shape& s) {
  const int R = s.g * s.Lo;
  return dtype == SNAP_BF16 && s.d_qk == D && (R == 128 || R == 256) && encode_tiled_fn() != nullptr;
}

// Candidate splits.  Every CTA takes the same number of candidate tiles (the chunk), whatever the
// prompt it works on, and the chunk is the smallest for which the CTAs of the launch fit whole
// waves of one CTA per SM -- one wave unless there are more (prompt, KV head) pairs than SMs.
// Long CTAs pay their set-up (query block, tensor memory, barriers) once per SM (measured: 171 ->
// 157 us for a 77k-token prompt, 242 -> 234 us at 128k, against two CTAs per SM in sequence), and
// equal ones leave no tail in a ragged batch.  Returns the splits of the longest prompt (the grid's x
// extent and the stride of the per-split statistics) and the chunk.
int score_umma_nsplit(const Shape& s, const int* le, int n_scored, int sm_count, int* chunk_tiles) {
  int max_tiles = 1;
  for (int i = 0; i < n_scored; ++i) max_tiles = max_tiles > (le[i] + TN - 1) / TN ? max_tiles : (le[i] + TN - 1) / TN;
  auto ctas = [&](int c) {
    long long n = 0;
    for (int i = 0; i < n_scored; ++i) n += ((le[i] + TN - 1) / TN + c - 1) / c;
    return n * s.Hkv;
  };
  int c = max_tiles;
  if (const int v = option(SNAP_OPT_SCORE_NSPLIT)) {            // tuning aid: splits of the longest prompt
    c = (max_tiles + v - 1) / v;
  } else {
    const long long nz = (long long)n_scored * s.Hkv;
    const long long target = (nz + sm_count - 1) / sm_count * sm_count;
    int lo = 1, hi = max_tiles;                                 // smallest chunk whose CTAs fit the target
    while (lo < hi) {
      const int mid = (lo + hi) / 2;
      if (ctas(mid) <= target) hi = mid; else lo = mid + 1;
    }
    c = lo;
  }
  if ((max_tiles + c - 1) / c > 512) c = (max_tiles + 511) / 512;
  if (c < 1) c = 1;
  *chunk_tiles = c;
  return (max_tiles + c - 1) / c;
}

cudaError_t launch_score_umma(const Shape& s, const SeqBatch& b, const void* q_obs, const KVSource& src,
                              const ScoreBuffers& buf, uint32_t* status, cudaStream_t st) {
  if (b.n_scored == 0) return cudaSuccess;
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return cudaErrorNotSupported;
  UmmaArgs a;
  a.Hq = s.Hq; a.Hkv = s.Hkv; a.g = s.g; a.Lo = s.Lo; a.Ls = s.Ls; a.Lr = s.Lr; a.R = s.g * s.Lo;
  a.scale_log2 = s.scale * 1.4426950408889634f;
  a.b = b; a.buf = buf; a.status = status;

  CUtensorMap tq, tk;
  const cuuint32_t estr2[2] = {1, 1}, estr3[3] = {1, 1, 1};
  {
    const cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)(b.first_seq + b.n) * s.Hq * s.Lo};
    const cuuint64_t strides[1] = {(cuuint64_t)D * 2};
    const cuuint32_t box[2] = {64, 128};
    if (enc(&tq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(q_obs), dims, strides, box, estr2,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
  }
  {
    long long tokens = 0;
    for (int i = 0; i < b.n; ++i) tokens = tokens > (long long)b.tok_off[i] + b.len[i] ? tokens : (long long)b.tok_off[i] + b.len[i];
    const long long head_stride = src.k_head_stride >= D ? src.k_head_stride : D;
    const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)s.Hkv, (cuuint64_t)tokens};
    const cuuint64_t strides[2] = {(cuuint64_t)head_stride * 2, (cuuint64_t)src.k_tok_stride * 2};
    const cuuint32_t box[3] = {64, 1, (cuuint32_t)TN};
    if (enc(&tk, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(src.k), dims, strides, box, estr3,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
  }
  static SmemLimit limit1 = {}, limit2 = {};
  if (cudaError_t e = ensure_dyn_smem(score_umma_kernel<1>, smem_bytes(1), limit1)) return e;
  if (cudaError_t e = ensure_dyn_smem(score_umma_kernel<2>, smem_bytes(2), limit2)) return e;
  const int nz = b.n_scored * s.Hkv;
  dim3 grid(buf.nsplit, nz);
  if (!buf.ext_mu) {                                          // Eq. 4's normalisers: pass 1, unless the caller has them
    if (launch_pdl(score_umma_kernel<1>, grid, dim3(NTHREADS), smem_bytes(1), st, a, tq, tk) != cudaSuccess) return cudaGetLastError();
    count_launch();
    cudaError_t e = launch_score_combine_log2(buf, nz, a.R, st);
    if (e != cudaSuccess) return e;
  }
  if (launch_pdl(score_umma_kernel<2>, grid, dim3(NTHREADS), smem_bytes(2), st, a, tq, tk) != cudaSuccess) return cudaGetLastError();
  count_launch();
  return cudaGetLastError();
}

}  // namespace snap
