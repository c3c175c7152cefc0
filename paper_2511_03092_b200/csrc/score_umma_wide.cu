// Observation-window scores (Eq. 4 -> Eq. 1) on tcgen05 for wide rows and many window rows --
// the latent-attention shape: 128 query heads x Lo rows (4096 window rows) against 576-wide keys;
// also every other bf16 shape with rows of 64 to 576 dims in steps of 64 (a partly filled last
// block of window rows is masked).
//
// Same roles as the 128-wide kernel (TMA producer warp, single-thread MMA issuer, eight epilogue
// warps reading TMEM), but the contraction dimension is streamed: a CTA keeps its 128-row query
// block resident in shared memory (one 16 KB swizzled slab per 64 dims) and, for every candidate
// tile, pulls the keys through a ring of stages (whatever fits beside the query block) one 64-dim
// slab at a time, accumulating in tensor memory; two accumulator buffers let the next tile's MMAs
// overlap the epilogue of the current one.
// With an even number of row blocks two CTAs with adjacent row blocks form a cluster and share every
// key tile (tcgen05 cta_group::2): each loads half of the tile's rows into its own shared memory,
// the even CTA issues M = 256 instructions over both, and each CTA finds its 128 rows of the
// accumulator in its own tensor memory -- half the L2-to-SM traffic per flop, which is what bounds
// the single-CTA form.  grid = (2 x candidate splits, row blocks / 2, prompts x KV heads) then;
// otherwise (candidate splits, row blocks, prompts x KV heads).
//   pass 1  M = 128 query rows, N = 256 candidates; thread = query row; the two epilogue groups
//           take 128 candidates each and their (reference max, sum) pairs are merged at the end.
//   pass 2  single CTAs: the same MMAs (an N = 128 instruction would occupy the tensor pipe almost as long
//           for half the work); thread = query row scales its row by exp2(-(m_i + log2 l_i)) and the 128
//           rows are summed per candidate with a transposing shuffle reduction and one shared-memory step.
//           Pairs: the operands are swapped -- M = 256 candidates (each CTA's own 128 of the tile), N = the
//           256 window rows of the pair's two row blocks -- so thread = candidate sums its own columns
//           and only the two epilogue groups' halves meet in shared memory.
//           Either way the per-row-group partial column sums go to scratch and a small kernel adds the
//           row groups in a fixed order (deterministic, no atomics).
// Every mbarrier wait is bounded; a wait that runs out raises SNAP_DEV_WAIT_TIMEOUT.
#include <cstdlib>

#include "snap_internal.cuh"
#include "umma_helpers.cuh"

namespace snap {
namespace {

using namespace umma;

constexpr int NTHREADS = 320, MAXNS = 6, MAXNS_PAIR = 8, STAGE_B = 32768, QH_B = 16384, MAXH = 9;

struct WideArgs {
  int Hq, Hkv, g, Lo, Ls, Lr, R, NH, RB;
  int RBC;               // row groups with a partial column sum each: RB, or RB / 2 when CTAs are paired
  int NS;                // key-slab stages: as many as fit beside the query block (2..MAXNS)
  float scale_log2;
  SeqBatch b;
  ScoreBuffers buf;
  float* cpart;          // [nz][RB][c_stride] partial column sums of pass 2
  uint32_t* status;
};

// PAIR: two CTAs with adjacent row blocks form a cluster and share every key tile: each loads one
// half of the tile's rows and the even CTA issues M = 256 instructions over both (cta_group::2).
template <int PASS, bool PAIR>
__global__ void __launch_bounds__(NTHREADS, 1)
score_umma_wide_kernel(const WideArgs a, const __grid_constant__ CUtensorMap tmap_q,
                       const __grid_constant__ CUtensorMap tmap_k) {
  constexpr int TNP = 256;                                    // candidates per tile
  constexpr int STG = PAIR ? STAGE_B / 2 : STAGE_B;           // bytes of a key slab held by this CTA
  const uint32_t crank = PAIR ? cluster_rank() : 0u;          // 0: issues the pair's MMAs
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int NH = a.NH, NS = a.NS;
  unsigned char* Qs = smem;                                   // [NH][128 rows][128 B]
  unsigned char* Ks = Qs + NH * QH_B;                         // [NS][256 rows (pair: this CTA's 128)][128 B]
  float* mu_s = reinterpret_cast<float*>(Ks + NS * STG);      // [128] pass 2: m_i + log2 l_i of this row block
  float2* xch = reinterpret_cast<float2*>(mu_s + 128);        // [128] exchange between the epilogue groups
  float* red = reinterpret_cast<float*>(xch + 128);           // [2 tile parities][2 groups][4 warps][128] pass-2 column partials
  // full[NS] empty[NS] tfull[2] tempty[2] qfull; in a pair the issuing CTA's full and qfull barriers count
  // the bytes of both CTAs' loads
  uint64_t* bars = reinterpret_cast<uint64_t*>(red + 2 * 2 * 4 * 128);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * NS + 5);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // a pair is two consecutive CTAs along x: grid = (2 x splits, row blocks / 2, prompts x KV heads) then, so that
  // CTAs that run at the same time still work on different candidate ranges
  const int rb = PAIR ? 2 * blockIdx.y + (blockIdx.x & 1) : blockIdx.y, split = PAIR ? blockIdx.x >> 1 : blockIdx.x;
  const int z = blockIdx.z, si = z / a.Hkv, kvh = z % a.Hkv;
  const int seq = a.b.seq_of_score[si];
  const int Le = a.b.len[seq] - a.Ls - a.Lr;
  const int R = a.R;
  const int ntiles = (Le + TNP - 1) / TNP;
  const int t0 = (int)((long long)ntiles * split / a.buf.nsplit);
  const int t1 = (int)((long long)ntiles * (split + 1) / a.buf.nsplit);
  const int nt = t1 - t0;

  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8 * s; };
  auto empty_bar = [&](int s) { return bar0 + 8 * (NS + s); };
  auto tfull_bar = [&](int b) { return bar0 + 8 * (2 * NS + b); };
  auto tempty_bar = [&](int b) { return bar0 + 8 * (2 * NS + 2 + b); };
  const uint32_t qfull_bar = bar0 + 8 * (2 * NS + 4);
  auto bwait = [&](uint32_t bar, unsigned parity) { return mbar_wait(bar, parity, abort_flag); };

  if (tid == 0) {
    *abort_flag = 0;
    for (int s = 0; s < NS; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), PAIR ? 16 : 8); }
    mbar_init(qfull_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (PASS == 2 && tid < (PAIR ? 256 : 128)) {
    // rows past the group's last one (a partly filled row block) get an infinite offset: weight 0
    // (a pair keeps the offsets of both its row blocks, negated, in the region `red`)
    const int row = (PAIR ? (rb & ~1) : rb) * 128 + tid;
    float mu = INFINITY;
    if (row < a.R) {
      if (a.buf.ext_mu) {                                      // [prompt][Hq][Lo]: a KV head's rows are consecutive
        mu = a.buf.ext_mu[((long long)(a.b.first_seq + seq) * a.Hq + kvh * a.g) * a.Lo + row];
      } else {
        const float2 st = a.buf.stats[(long long)z * a.R + row];
        mu = st.x - log2f(st.y);
      }
    }
    if (PAIR) red[tid] = -mu;
    else mu_s[tid] = mu;
  }
  if (warp == 0) {
    if (PAIR) {                                                // both CTAs of the pair, same warp, same slot
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  fence_before();
  __syncthreads();
  if (PAIR) cluster_barrier();                                 // the other CTA's barriers exist before anything arrives on them
  fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int eg = warp >= 2 ? (warp - 2) >> 2 : 0;             // epilogue group
  const int lrow = 32 * (warp & 3) + lane;                    // accumulator row = TMEM lane
  float m_ref = -INFINITY, l_sum = 0.f;                       // pass 1: statistics of query row rb*128 + lrow

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    // (stage index and phase are carried along: the issuing threads' instruction chains bound these
    // kernels, so neither loop divides, and the descriptors' constant parts are built once)
    if (lane == 0 && nt > 0) {
      const int row0 = ((a.b.first_seq + seq) * a.Hq + kvh * a.g) * a.Lo + rb * 128;
      int tok = a.b.tok_off[seq] + a.Ls + t0 * TNP + (PAIR ? (int)crank * 128 : 0);
      bool ok = true;
      // in a pair both CTAs' bytes are counted on the issuing CTA's barriers, which that CTA arms for both
      const uint32_t lead = PAIR ? map_to_rank(bar0, 0) - bar0 : 0u;   // offset to the same barrier in the issuing CTA
      if (PAIR) {
        if (crank == 0) mbar_expect_tx(qfull_bar, 2u * (unsigned)NH * QH_B);
        for (int h = 0; h < NH; ++h) tma_load_2d_pair(smem_u32(Qs) + h * QH_B, &tmap_q, h * 64, row0, qfull_bar + lead);
      } else {
        mbar_expect_tx(qfull_bar, (unsigned)NH * QH_B);
        for (int h = 0; h < NH; ++h) tma_load_2d(smem_u32(Qs) + h * QH_B, &tmap_q, h * 64, row0, qfull_bar);
      }
      int s = 0;
      unsigned ph = 1u;                                        // parity of the "stage is free" phase awaited next
      uint32_t dst = smem_u32(Ks), fb = full_bar(0);
      for (int it = 0; it < nt && ok; ++it, tok += TNP)
        for (int h = 0; h < NH; ++h) {
          if (!bwait(fb + 8 * NS, ph)) { *abort_flag = 1; ok = false; break; }
          if (PAIR) {
            if (crank == 0) mbar_expect_tx(fb, 2u * (unsigned)STG);
            tma_load_3d_pair(dst, &tmap_k, h * 64, kvh, tok, fb + lead);
          } else {
            mbar_expect_tx(fb, (unsigned)STG);
            tma_load_3d(dst, &tmap_k, h * 64, kvh, tok, fb);
          }
          if (++s == NS) { s = 0; ph ^= 1u; dst = smem_u32(Ks); fb = full_bar(0); }
          else { dst += STG; fb += 8; }
        }
      if (PAIR) {
        // the issuing CTA's commits arrive on this CTA's barriers asynchronously: take the last ones in
        // before leaving, so that none lands in a CTA that has exited
        const int total = nt * NH;
        for (int q = total > NS ? total - NS : 0; q < total && ok; ++q)
          ok = bwait(empty_bar(q % NS), (unsigned)(q / NS) & 1u);
        if (!ok) *abort_flag = 1;
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0 && nt > 0 && crank == 0) {
      const uint32_t idesc = idesc_bf16(PAIR ? 256 : 128, 256);
      const uint64_t qdesc0 = smem_desc(smem_u32(Qs)), kdesc0 = smem_desc(smem_u32(Ks));
      const uint32_t peer = PAIR ? map_to_rank(bar0, 1) - bar0 : 0u;   // offset to the same barrier in the other CTA
      bool ok = mbar_wait(qfull_bar, 0u, abort_flag);
      int s = 0;
      unsigned ph = 0u;                                        // parity of the "slab has landed" phase awaited next
      uint64_t kdesc = kdesc0;
      uint32_t fb = full_bar(0);
      for (int it = 0; it < nt && ok; ++it) {
        const int b = it & 1;
        ok = bwait(tempty_bar(b), ((unsigned)(it >> 1) & 1u) ^ 1u);
        fence_after();
        uint64_t qdesc = qdesc0;
        const uint32_t acc = tmem_base + b * 256;
        for (int h = 0; h < NH && ok; ++h, qdesc += QH_B >> 4) {
          ok = mbar_wait(fb, ph, abort_flag);
          if (!ok) break;
          if (PASS == 2 && PAIR) mma_slab4<PAIR>(acc, kdesc, qdesc, idesc, h != 0);   // candidates on M, window rows on N
          else mma_slab4<PAIR>(acc, qdesc, kdesc, idesc, h != 0);
          // the slab may be refilled once these MMAs have read it (in both CTAs of a pair)
          if (PAIR) { mma_commit_pair(fb + 8 * NS); mma_commit_pair(fb + 8 * NS + peer); }
          else mma_commit(fb + 8 * NS);
          if (++s == NS) { s = 0; ph ^= 1u; kdesc = kdesc0; fb = full_bar(0); }
          else { kdesc += STG >> 4; fb += 8; }
        }
        if (ok) {                                              // accumulator buffer complete
          if (PAIR) { mma_commit_pair(tfull_bar(b)); mma_commit_pair(tfull_bar(b) + peer); }
          else mma_commit(tfull_bar(b));
        }
      }
      if (!ok) *abort_flag = 1;
    }
  } else {
    // ---------------- epilogue warps ----------------
    const uint32_t lane_addr = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16);
    bool ok = true;
    auto release_acc = [&](int b) {                            // the accumulator buffer may be overwritten
      if (PAIR && crank != 0) mbar_arrive_remote(map_to_rank(tempty_bar(b), 0));
      else mbar_arrive(tempty_bar(b));
    };
    const float neg_mu = PASS == 2 && !PAIR ? -mu_s[lrow] : 0.f;   // pass 2, single CTAs: this thread's row offset (-inf for a padding row)
    for (int it = 0; it < nt; ++it) {
      const int b = it & 1;
      const bool landed = bwait(tfull_bar(b), (unsigned)(it / 2) & 1u);
      if (!landed) {
        *abort_flag = 1;
        ok = false;
        if (PASS == 1) break;                                  // pass 2 leaves through the group barrier below
      }
      fence_after();
      uint32_t ra[16], rb16[16];
      if (PASS == 1) {
        const uint32_t col0 = lane_addr + b * 256 + eg * 128;
        const int cand0 = (t0 + it) * TNP + eg * 128;         // first candidate of this group's columns
        const bool full_tile = cand0 + 128 <= Le;
        // sum of exp2 over this group's 128 columns relative to reference `ref`
        auto sweep = [&](float ref, bool want_max, float& vmax) -> float {
          float s4[4] = {0.f, 0.f, 0.f, 0.f};
          tmem_ld16_issue(col0, ra);
#pragma unroll
          for (int c = 0; c < 8; c += 2) {
            tmem_ld16_wait(ra);
            tmem_ld16_issue(col0 + 16 * (c + 1), rb16);
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float v = __uint_as_float(ra[i]) * a.scale_log2;
              const bool in = full_tile || cand0 + 16 * c + i < Le;
              if (want_max) { if (in) vmax = fmaxf(vmax, v); }
              else s4[i & 3] += in ? fast_exp2(v - ref) : 0.f;
            }
            tmem_ld16_wait(rb16);
            if (c + 2 < 8) tmem_ld16_issue(col0 + 16 * (c + 2), ra);
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float v = __uint_as_float(rb16[i]) * a.scale_log2;
              const bool in = full_tile || cand0 + 16 * (c + 1) + i < Le;
              if (want_max) { if (in) vmax = fmaxf(vmax, v); }
              else s4[i & 3] += in ? fast_exp2(v - ref) : 0.f;
            }
          }
          return (s4[0] + s4[1]) + (s4[2] + s4[3]);
        };
        // the common case (a tile wholly inside the candidates, reference up to date) with two-wide
        // packed arithmetic: half an issue slot per element for the multiply-add and for the sum
        auto sweep_full = [&](float ref) -> float {
          u64 acc[2] = {pack2(0.f, 0.f), pack2(0.f, 0.f)};
          const u64 sc2 = pack2(a.scale_log2, a.scale_log2), nr2 = pack2(-ref, -ref);
          tmem_ld16_issue(col0, ra);
#pragma unroll
          for (int c = 0; c < 8; c += 2) {
            tmem_ld16_wait(ra);
            tmem_ld16_issue(col0 + 16 * (c + 1), rb16);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const u64 x = fma2(pack2(__uint_as_float(ra[2 * i]), __uint_as_float(ra[2 * i + 1])), sc2, nr2);
              acc[i & 1] = add2(acc[i & 1], pack2(fast_exp2(lo2(x)), fast_exp2(hi2(x))));
            }
            tmem_ld16_wait(rb16);
            if (c + 2 < 8) tmem_ld16_issue(col0 + 16 * (c + 2), ra);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const u64 x = fma2(pack2(__uint_as_float(rb16[2 * i]), __uint_as_float(rb16[2 * i + 1])), sc2, nr2);
              acc[i & 1] = add2(acc[i & 1], pack2(fast_exp2(lo2(x)), fast_exp2(hi2(x))));
            }
          }
          return (lo2(acc[0]) + hi2(acc[0])) + (lo2(acc[1]) + hi2(acc[1]));
        };
        float dummy = 0.f;
        float sum = full_tile ? sweep_full(m_ref) : sweep(m_ref, false, dummy);
        // a logit far above the reference (or the first tile): refresh it; the TMEM loads are
        // warp-collective, so the whole warp takes the branch if any row needs it
        if (__any_sync(0xffffffffu, !(sum < 65536.f))) {
          float vmax = -INFINITY;
          (void)sweep(0.f, true, vmax);
          const float mn = fmaxf(m_ref, vmax);
          sum = 0.f;
          if (mn != -INFINITY) {
            l_sum *= m_ref == -INFINITY ? 0.f : fast_exp2(m_ref - mn);
            m_ref = mn;
          }
          const float s2 = sweep(mn == -INFINITY ? 0.f : mn, false, dummy);
          if (mn != -INFINITY) sum = s2;
        }
        l_sum += sum;
      } else if (PAIR) {
        // Pair: the operands are swapped, so thread = candidate (this CTA's 128 of the tile's 256) and the columns are
        // the 256 window rows of the pair's two row blocks, one block per epilogue group.  The weights
        // exp2(s - m_i - log2 l_i) are summed along the thread's own columns: no exchange between threads, only
        // the two groups' halves are added through shared memory.
        const uint32_t col0 = lane_addr + b * 256 + eg * 128;
        const int cand = (t0 + it) * TNP + (int)crank * 128 + lrow;
        const float* nmu = red + eg * 128;                       // -(m_i + log2 l_i) of this group's rows
        const u64 sc2 = pack2(a.scale_log2, a.scale_log2);
        u64 acc2[2] = {pack2(0.f, 0.f), pack2(0.f, 0.f)};
        if (landed) {
          tmem_ld16_issue(col0, ra);
#pragma unroll
          for (int c = 0; c < 8; c += 2) {
            tmem_ld16_wait(ra);
            tmem_ld16_issue(col0 + 16 * (c + 1), rb16);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const ulonglong2 m4 = *reinterpret_cast<const ulonglong2*>(nmu + 16 * c + 4 * i);   // the same address in every lane
              const u64 x0 = fma2(pack2(__uint_as_float(ra[4 * i]), __uint_as_float(ra[4 * i + 1])), sc2, m4.x);
              const u64 x1 = fma2(pack2(__uint_as_float(ra[4 * i + 2]), __uint_as_float(ra[4 * i + 3])), sc2, m4.y);
              acc2[0] = add2(acc2[0], pack2(fast_exp2(lo2(x0)), fast_exp2(hi2(x0))));
              acc2[1] = add2(acc2[1], pack2(fast_exp2(lo2(x1)), fast_exp2(hi2(x1))));
            }
            tmem_ld16_wait(rb16);
            if (c + 2 < 8) tmem_ld16_issue(col0 + 16 * (c + 2), ra);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const ulonglong2 m4 = *reinterpret_cast<const ulonglong2*>(nmu + 16 * (c + 1) + 4 * i);
              const u64 x0 = fma2(pack2(__uint_as_float(rb16[4 * i]), __uint_as_float(rb16[4 * i + 1])), sc2, m4.x);
              const u64 x1 = fma2(pack2(__uint_as_float(rb16[4 * i + 2]), __uint_as_float(rb16[4 * i + 3])), sc2, m4.y);
              acc2[0] = add2(acc2[0], pack2(fast_exp2(lo2(x0)), fast_exp2(hi2(x0))));
              acc2[1] = add2(acc2[1], pack2(fast_exp2(lo2(x1)), fast_exp2(hi2(x1))));
            }
          }
        }
        fence_before();                                        // the accumulator buffer is free again
        __syncwarp();
        if (lane == 0) release_acc(b);
        const float sum = (lo2(acc2[0]) + hi2(acc2[0])) + (lo2(acc2[1]) + hi2(acc2[1]));
        float* gx = reinterpret_cast<float*>(xch) + (it & 1) * 128;   // double-buffered by tile parity: one barrier per tile
        if (eg == 1) gx[lrow] = sum;
        unsigned stop;                                         // barrier over both groups + agreement on giving up
        asm volatile(
            "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
            "bar.red.or.pred p, 1, 256, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(stop) : "r"((unsigned)(!landed || *abort_flag)) : "memory");
        if (eg == 0 && !stop && cand < Le)
          a.cpart[((long long)z * a.RBC + (rb >> 1)) * a.buf.c_stride + cand] = sum + gx[lrow];
        if (stop) { *abort_flag = 1; ok = false; }
      } else {
        // thread = query row; this group's 128 candidates of the tile.  The weights exp2(s - m_i - log2 l_i)
        // are summed over the 128 rows of the block: a transposing shuffle reduction inside each warp (every
        // step halves the values a lane holds), then over the group's four warps through shared memory.
        const uint32_t col0 = lane_addr + b * 256 + eg * 128;
        const int cand0 = (t0 + it) * TNP + eg * 128;
        float v[128];
        const u64 sc2 = pack2(a.scale_log2, a.scale_log2), nmu2 = pack2(neg_mu, neg_mu);
        if (landed) {
          tmem_ld16_issue(col0, ra);
#pragma unroll
          for (int c = 0; c < 8; c += 2) {
            tmem_ld16_wait(ra);
            tmem_ld16_issue(col0 + 16 * (c + 1), rb16);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const u64 x = fma2(pack2(__uint_as_float(ra[2 * i]), __uint_as_float(ra[2 * i + 1])), sc2, nmu2);
              v[16 * c + 2 * i] = fast_exp2(lo2(x));
              v[16 * c + 2 * i + 1] = fast_exp2(hi2(x));
            }
            tmem_ld16_wait(rb16);
            if (c + 2 < 8) tmem_ld16_issue(col0 + 16 * (c + 2), ra);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const u64 x = fma2(pack2(__uint_as_float(rb16[2 * i]), __uint_as_float(rb16[2 * i + 1])), sc2, nmu2);
              v[16 * (c + 1) + 2 * i] = fast_exp2(lo2(x));
              v[16 * (c + 1) + 2 * i + 1] = fast_exp2(hi2(x));
            }
          }
        } else {
#pragma unroll
          for (int i = 0; i < 128; ++i) v[i] = 0.f;
        }
        fence_before();                                        // the accumulator buffer is free again
        __syncwarp();
        if (lane == 0) release_acc(b);
#pragma unroll
        for (int bit = 16, width = 64; bit >= 1; bit >>= 1, width >>= 1) {
          const bool upper = (lane & bit) != 0;
#pragma unroll
          for (int e = 0; e < width; ++e) {
            const float send = upper ? v[e] : v[e + width];
            const float keep = upper ? v[e + width] : v[e];
            v[e] = keep + __shfl_xor_sync(0xffffffffu, send, bit);
          }
        }
        // the lane now holds the sums over its warp's 32 rows of four consecutive candidates
        const int colbase = ((lane >> 4) & 1) * 64 + ((lane >> 3) & 1) * 32 + ((lane >> 2) & 1) * 16 + ((lane >> 1) & 1) * 8 +
                            (lane & 1) * 4;
        float* rg = red + ((it & 1) * 2 + eg) * 4 * 128;       // double-buffered by tile parity: one barrier per tile
        *reinterpret_cast<float4*>(rg + (warp & 3) * 128 + colbase) = make_float4(v[0], v[1], v[2], v[3]);
        unsigned stop;                                         // barrier over the group's 4 warps + agreement on giving up
        asm volatile(
            "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
            "bar.red.or.pred p, %2, 128, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(stop) : "r"((unsigned)(!landed || *abort_flag)), "r"(1 + eg) : "memory");
        if (!stop && cand0 + lrow < Le)
          a.cpart[((long long)z * a.RBC + rb) * a.buf.c_stride + cand0 + lrow] =
              (rg[lrow] + rg[128 + lrow]) + (rg[256 + lrow] + rg[384 + lrow]);
        if (stop) { *abort_flag = 1; ok = false; }
      }
      if (PASS == 1) {
        fence_before();
        __syncwarp();
        if (lane == 0) release_acc(b);
      }
      if (!ok) break;
    }
    if (!ok) *abort_flag = 1;
    if (PASS == 1 && eg == 1) xch[lrow] = make_float2(m_ref, l_sum);
  }

  fence_before();
  __syncthreads();
  fence_after();
  if (PASS == 1 && warp >= 2 && eg == 0 && rb * 128 + lrow < R) {   // the two groups took different candidates of each tile
    const float2 o = xch[lrow];
    merge_ml(m_ref, l_sum, o.x, o.y);
    a.buf.part_stats[((long long)z * a.buf.nsplit + split) * R + rb * 128 + lrow] = make_float2(m_ref, l_sum);
  }
  if (PAIR) cluster_barrier();                                 // nobody leaves while the other CTA may still signal it
  if (warp == 0) {
    if (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
  if (tid == 0 && *abort_flag && a.status) atomicOr(a.status, SNAP_DEV_WAIT_TIMEOUT);
}

// C[z][j] = sum over the row blocks of the partial column sums, in a fixed order.
__global__ void score_rowblock_reduce_kernel(const float* __restrict__ cpart, float* __restrict__ C, int RB,
                                             int c_stride, SeqBatch b, int Hkv, int Ls, int Lr) {
  const int z = blockIdx.y, si = z / Hkv;
  const int Le = b.len[b.seq_of_score[si]] - Ls - Lr;
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= Le) return;
  float s = 0.f;
  for (int rb = 0; rb < RB; ++rb) s += cpart[((long long)z * RB + rb) * c_stride + j];
  C[(long long)z * c_stride + j] = s;
}

size_t wide_smem_bytes(int NH, int NS, bool pair) {
  return (size_t)NH * QH_B + NS * (pair ? STAGE_B / 2 : STAGE_B) + 128 * sizeof(float) + 128 * sizeof(float2) +
         2 * 2 * 4 * 128 * sizeof(float) + (2 * NS + 5) * 8 + 16 + 1024;
}

// Option SNAP_OPT_WIDE_STAGES caps the ring depth (tuning aid).
int wide_stages(int NH, bool pair) {
  int ns = pair ? MAXNS_PAIR : MAXNS;
  if (const int v = option(SNAP_OPT_WIDE_STAGES))
    if (v >= 2 && v < ns) ns = v;
  while (ns > 2 && wide_smem_bytes(NH, ns, pair) > 227u * 1024u) --ns;
  return ns;
}

// CTA pairs need an even number of row blocks; option SNAP_OPT_SCORE_KERNEL = 3 keeps single CTAs.
bool wide_pairs(int RB) { return RB % 2 == 0 && option(SNAP_OPT_SCORE_KERNEL) != 3; }

template <int PASS, bool PAIR>
cudaError_t launch_wide(dim3 grid, size_t smem, cudaStream_t st, const WideArgs& a, const CUtensorMap& tq, const CUtensorMap& tk) {
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = PAIR ? 2 : 1;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = grid;
  lc.blockDim = dim3(NTHREADS);
  lc.dynamicSmemBytes = smem;
  lc.stream = st;
  lc.attrs = attr;
  lc.numAttrs = 1;
  count_launch();
  return cudaLaunchKernelEx(&lc, score_umma_wide_kernel<PASS, PAIR>, a, tq, tk);
}

}  // namespace

bool score_umma_wide_supported(int dtype, const Shape& s) {
  const int R = s.g * s.Lo;
  return dtype == SNAP_BF16 && s.d_qk % 64 == 0 && s.d_qk / 64 <= MAXH && R >= 1 &&
         umma::encode_tiled_fn() != nullptr;
}

int score_umma_wide_row_blocks(const Shape& s) { return (s.g * s.Lo + 127) / 128; }

// Candidate splits: about two CTAs per SM in sequence over (splits x row blocks x prompts x KV heads).
int score_umma_wide_nsplit(const Shape& s, int n_scored, int max_le, int sm_count) {
  const int tiles = (max_le + 255) / 256;
  const long long base = (long long)n_scored * s.Hkv * score_umma_wide_row_blocks(s);
  if (const int v = option(SNAP_OPT_SCORE_NSPLIT))              // tuning aid
    return v < tiles ? (v < 512 ? v : 512) : tiles;
  long long ns = (2LL * sm_count + base / 2) / base;
  if (ns > tiles) ns = tiles;
  if (ns > 512) ns = 512;
  if (ns < 1) ns = 1;
  return (int)ns;
}

cudaError_t launch_score_umma_wide(const Shape& s, const SeqBatch& b, const void* q_obs, const KVSource& src,
                                   const ScoreBuffers& buf, float* cpart, uint32_t* status, cudaStream_t st) {
  if (b.n_scored == 0) return cudaSuccess;
  umma::EncodeTiledFn enc = umma::encode_tiled_fn();
  if (!enc) return cudaErrorNotSupported;
  WideArgs a;
  a.Hq = s.Hq; a.Hkv = s.Hkv; a.g = s.g; a.Lo = s.Lo; a.Ls = s.Ls; a.Lr = s.Lr; a.R = s.g * s.Lo;
  a.NH = s.d_qk / 64; a.RB = (a.R + 127) / 128;
  const bool pair = wide_pairs(a.RB);
  a.RBC = pair ? a.RB / 2 : a.RB;
  a.NS = wide_stages(a.NH, pair);
  a.scale_log2 = s.scale * 1.4426950408889634f;
  a.b = b; a.buf = buf; a.cpart = cpart; a.status = status;

  CUtensorMap tq, tk1;
  const cuuint32_t estr2[2] = {1, 1}, estr3[3] = {1, 1, 1};
  {
    const cuuint64_t dims[2] = {(cuuint64_t)s.d_qk, (cuuint64_t)(b.first_seq + b.n) * s.Hq * s.Lo};
    const cuuint64_t strides[1] = {(cuuint64_t)s.d_qk * 2};
    const cuuint32_t box[2] = {64, 128};
    if (enc(&tq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(q_obs), dims, strides, box, estr2,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
  }
  long long tokens = 0;
  for (int i = 0; i < b.n; ++i) tokens = tokens > (long long)b.tok_off[i] + b.len[i] ? tokens : (long long)b.tok_off[i] + b.len[i];
  const long long head_stride = src.k_head_stride >= s.d_qk ? src.k_head_stride : s.d_qk;
  const cuuint64_t kdims[3] = {(cuuint64_t)s.d_qk, (cuuint64_t)s.Hkv, (cuuint64_t)tokens};
  const cuuint64_t kstrides[2] = {(cuuint64_t)head_stride * 2, (cuuint64_t)src.k_tok_stride * 2};
  const cuuint32_t kbox[3] = {64, 1, pair ? 128u : 256u};      // one 64-dim slab of a 256-candidate tile (pair: this CTA's half)
  if (enc(&tk1, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(src.k), kdims, kstrides, kbox, estr3,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  const size_t smem = wide_smem_bytes(a.NH, a.NS, pair);
  static SmemLimit limit1 = {}, limit2 = {}, limit1p = {}, limit2p = {};
  if (pair) {
    if (cudaError_t e = ensure_dyn_smem(score_umma_wide_kernel<1, true>, smem, limit1p)) return e;
    if (cudaError_t e = ensure_dyn_smem(score_umma_wide_kernel<2, true>, smem, limit2p)) return e;
  } else {
    if (cudaError_t e = ensure_dyn_smem(score_umma_wide_kernel<1, false>, smem, limit1)) return e;
    if (cudaError_t e = ensure_dyn_smem(score_umma_wide_kernel<2, false>, smem, limit2)) return e;
  }
  const int nz = b.n_scored * s.Hkv;
  int max_le = 0;
  for (int i = 0; i < b.n; ++i)
    if (b.score_idx[i] >= 0) max_le = max_le > b.len[i] - s.Ls - s.Lr ? max_le : b.len[i] - s.Ls - s.Lr;
  const dim3 grid = pair ? dim3(2 * buf.nsplit, a.RB / 2, nz) : dim3(buf.nsplit, a.RB, nz);
  if (!buf.ext_mu) {                                          // Eq. 4's normalisers: pass 1, unless the caller has them
    cudaError_t e = pair ? launch_wide<1, true>(grid, smem, st, a, tq, tk1) : launch_wide<1, false>(grid, smem, st, a, tq, tk1);
    if (e != cudaSuccess) return e;
    e = launch_score_combine_log2(buf, nz, a.R, st);
    if (e != cudaSuccess) return e;
  }
  if (cudaError_t e = pair ? launch_wide<2, true>(grid, smem, st, a, tq, tk1) : launch_wide<2, false>(grid, smem, st, a, tq, tk1))
    return e;
  score_rowblock_reduce_kernel<<<dim3((max_le + 255) / 256, nz), 256, 0, st>>>(cpart, buf.C, a.RBC, buf.c_stride, b,
                                                                            s.Hkv, s.Ls, s.Lr);
  count_launch();
  return cudaGetLastError();
}

}  // namespace snap
