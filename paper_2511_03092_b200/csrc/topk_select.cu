// Sequence-axis pooling and per-KV-head top-K (Eq. 2), one cluster of 8 CTAs per (prompt, KV head).
//
//   P[j] = pool_w(C)[j]  (1-D, stride 1, pad w/2; average divides by w over zero padding, max pads -inf)
//   keep the K largest P, ties to the lower index, and emit absolute positions in ascending order.
//
// Each CTA of the cluster owns a contiguous eighth of the candidates.  Selection is an
// 8-bit-digit radix select on the order-preserving integer image of P: four histogram passes
// narrow down the K-th largest key (the high bits that all keys share are found first with a
// cluster-wide min/max and skipped).  Histograms are per pair of warps in shared memory, summed
// per CTA, and every CTA sends its histogram to all eight CTAs with asynchronous remote stores
// that complete on the receiver's mbarrier (st.async): each CTA waits for its own eight arrivals,
// adds them up and finds the same digit as the others -- no broadcast and no cluster barrier per
// pass (a cluster barrier with release/acquire semantics costs about as much as the rest of a
// pass).  The only cluster barrier is the one that publishes the initialised mbarriers, and its
// wait is placed after the loads and the pooling.  Then an ordered compaction: every key above
// the threshold is taken, and of the keys equal to it the first ones in index order until K are
// reached; CTA offsets come from the per-CTA counts (exchanged the same way) -- no global
// atomics, deterministic output.  A CTA leaves only after it has received every message
// addressed to it, and nobody reads another CTA's shared memory, so no barrier is needed at the
// end either.
//
// Two kernels share that scheme.  The register-resident one (prompts up to 128k tokens, pooling
// kernels up to 17) gives every thread 16 consecutive candidates: it loads their score window
// once, pools it in registers, keeps the 16 keys in registers through all passes, and because
// thread order is index order one block scan places the whole slice.  The streaming one keeps
// pooled scores in scratch and handles any length.
// Prompts with at most K candidates keep them all and are not scored.
//
// For the double-precision refinement (topk_refine.cu) the emission step also records the band:
// every candidate whose pooled score lies within a relative distance of the threshold, with a
// flag saying whether the single-precision order selected it, and the number of candidates
// above the band.
#include <cooperative_groups.h>

#include "snap_internal.cuh"
#include "umma_helpers.cuh"

namespace cg = cooperative_groups;

namespace snap {
namespace {

constexpr int NT = 1024, NW = NT / 32, NH = NW / 2, CL = 8, MAXE = 16, MAXR = 8;
constexpr unsigned kInboxWaitLimit = 1u << 22;
constexpr int LIST_CAP = 64;

struct TopkArgs {
  int Hkv, Ls, Lr, K, w, pool_mode;
  SeqBatch b;
  ScoreBuffers buf;
  int* idx_out;      // [n][Hkv][K]
  uint32_t* status;
};

struct TopkShared {
  int hist[NH][256];                 // one histogram per pair of warps
  alignas(16) int inbox[2][CL][256]; // the eight CTA histograms of a pass, written by their owners (double buffered)
  alignas(16) int cta_bins[256];     // this CTA's histogram of the current pass
  alignas(8) unsigned minmax[CL][2]; // (smallest, largest) key of every CTA, written by its owner
  alignas(8) int counts[CL][2];      // (greater, equal) counts of every CTA, written by its owner
  alignas(16) unsigned list[LIST_CAP]; // the keys of the whole cluster that still match the prefix (short-cut below)
  unsigned long long bar[5];         // arrival of: histograms (two buffers), min/max, counts, list
  int warp_tot[NW + 1];
  unsigned prefix;
  int remaining;
  int sure;              // this CTA's candidates above the re-scoring band
  int failed;            // a bounded wait ran out
  int digit, alive;      // the digit chosen by the last pass and how many keys of the cluster carry it
  int list_n;            // keys this CTA has put on the list
};

// ---- messages between the CTAs of the cluster: remote stores that complete on the receiver's mbarrier ----
__device__ __forceinline__ void send4(uint32_t dst, uint32_t dst_bar, int4 v) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
               ::"r"(dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "r"(dst_bar) : "memory");
}
__device__ __forceinline__ void send1(uint32_t dst, uint32_t dst_bar, unsigned x) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];"
               ::"r"(dst), "r"(x), "r"(dst_bar) : "memory");
}
__device__ __forceinline__ void send2(uint32_t dst, uint32_t dst_bar, unsigned x, unsigned y) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.b32 [%0], {%1, %2}, [%3];"
               ::"r"(dst), "r"(x), "r"(y), "r"(dst_bar) : "memory");
}
// Bounded wait for the messages of one exchange; a wait that runs out raises SNAP_DEV_WAIT_TIMEOUT and
// CTA skips its emission (sh.failed).
__device__ __forceinline__ void inbox_wait(TopkShared& sh, int which, unsigned parity, uint32_t* status) {
  const uint32_t b = umma::smem_u32(&sh.bar[which]);
  for (unsigned it = 0; it < kInboxWaitLimit; ++it)
    if (umma::mbar_try_wait(b, parity)) return;
  sh.failed = 1;
  if (status) atomicOr(status, SNAP_DEV_WAIT_TIMEOUT);
}
// Thread 0 of every CTA: barriers ready for the first exchange.  Followed by cluster.barrier_arrive();
// the matching wait comes before the first message is sent.
__device__ __forceinline__ void inbox_init(TopkShared& sh) {
  if (threadIdx.x == 0) {
#pragma unroll
    for (int i = 0; i < 5; ++i) umma::mbar_init(umma::smem_u32(&sh.bar[i]), 1);
    sh.failed = 0;
    sh.list_n = 0;
    sh.alive = 0x7fffffff;
    sh.digit = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
}

__device__ __forceinline__ unsigned key_of(float x) {
  const unsigned u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float value_of(unsigned key) {
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// The band around the threshold key and where its members are recorded.
struct Band {
  RefineHead* head;
  BandEntry* entries;
  int cap;
  unsigned lo, hi;
};
__device__ __forceinline__ Band make_band(const TopkArgs& a, long long z, unsigned tau) {
  Band bd;
  bd.head = a.buf.ref.head ? a.buf.ref.head + z : nullptr;
  bd.entries = a.buf.ref.head ? a.buf.ref.band + z * a.buf.ref.cap : nullptr;
  bd.cap = a.buf.ref.cap;
  const float t = value_of(tau), dt = fabsf(t) * a.buf.ref.rel;
  bd.lo = key_of(t - dt);
  bd.hi = key_of(t + dt);
  return bd;
}
__device__ __forceinline__ void band_record(const Band& bd, unsigned key, int j, bool selected) {
  if (key < bd.lo || key > bd.hi) return;
  const int slot = atomicAdd(&bd.head->n_band, 1);
  if (slot < bd.cap) {
    BandEntry e;
    e.idx_flag = j | (selected ? (int)0x80000000u : 0);
    e.p32 = value_of(key);
    bd.entries[slot] = e;
  }
}
// Adds this thread's count of candidates above the band to the head's total: summed per warp, then per
// CTA in shared memory, one global atomic per CTA (hundreds of warps on one address serialise).
__device__ __forceinline__ void band_count_sure(const Band& bd, int n, int* cta_sum) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) n += __shfl_xor_sync(0xffffffffu, n, o);
  if ((threadIdx.x & 31) == 0 && n > 0) atomicAdd(cta_sum, n);
  __syncthreads();
  if (threadIdx.x == 0 && *cta_sum > 0) atomicAdd(&bd.head->n_sure, *cta_sum);
}
__device__ __forceinline__ void band_reset(const TopkArgs& a, long long z, int rank) {
  if (a.buf.ref.head && rank == 0 && threadIdx.x == 0) {
    RefineHead h = {};
    a.buf.ref.head[z] = h;       // ordered before every use by the cluster barriers of the select
  }
}

// Exclusive prefix sum of one int per thread over the whole CTA (thread order), plus the total.
__device__ __forceinline__ int block_exscan(int v, int* warp_tot, int& total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  if (lane == 31) warp_tot[wid] = inc;
  __syncthreads();
  if (wid == 0) {
    const int t = warp_tot[lane];
    int winc = t;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += n;
    }
    warp_tot[lane] = winc - t;
    if (lane == 31) warp_tot[NW] = winc;
  }
  __syncthreads();
  const int r = warp_tot[wid] + inc - v;
  total = warp_tot[NW];
  __syncthreads();
  return r;
}

// One histogram update: a predicated shared-memory reduction -- no branch, and nothing is returned, so
// the sixteen updates of a thread are seven instructions each and do not wait for one another.  (These
// loops run in all 32 warps of the SM's only CTA: they are bound by instruction issue, eight warps per
// scheduler.)
__device__ __forceinline__ void hist_add(int* warp_hist, unsigned key, unsigned mask, unsigned prefix, int shift,
                                         unsigned dmask) {
  const unsigned miss = (key & mask) ^ prefix;
  const uint32_t addr = umma::smem_u32(warp_hist) + (((key >> shift) & dmask) << 2);
  asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.u32 p, %1, 0;\n\t@p red.shared.add.u32 [%0], 1;\n\t}" ::"r"(addr), "r"(miss)
               : "memory");
}
// FULL: the thread owns all MAXE candidates (every thread but those of a slice's last warps).
template <bool FULL>
__device__ __forceinline__ void hist_keys(int* warp_hist, const unsigned (&keys)[16], int nmine, unsigned mask,
                                          unsigned prefix, int shift, unsigned dmask) {
#pragma unroll
  for (int k = 0; k < 16; ++k)
    if (FULL || k < nmine) hist_add(warp_hist, keys[k], mask, prefix, shift, dmask);
}
__device__ __forceinline__ void hist_clear(TopkShared& sh) {
  for (int i = threadIdx.x; i < NH * 256; i += NT) (&sh.hist[0][0])[i] = 0;
}

// Smallest and largest key of the cluster.  The bits above the highest bit in which they differ
// are common to every key and need no histogram pass (pooled scores share sign and most of the
// exponent, so the leading digit would otherwise put a whole warp on one counter).
// Returns the number of low bits still to be resolved; sets sh.prefix to the common high bits.
// Completes the cluster barrier that inbox_init started.
__device__ __forceinline__ int cluster_common_prefix(cg::cluster_group& cluster, TopkShared& sh, int rank, unsigned kmin,
                                                     unsigned kmax, int K, uint32_t* status) {
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
    kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
  }
  unsigned* mm = reinterpret_cast<unsigned*>(sh.cta_bins);         // [0..31] warp minima, [32..63] maxima
  if (lane == 0) { mm[wid] = kmin; mm[32 + wid] = kmax; }
  cluster.barrier_wait();                            // every CTA's mbarriers are initialised (and this CTA's mm is written)
  __syncthreads();
  if (wid == 0) {
    kmin = mm[lane]; kmax = mm[32 + lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
      kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
    }
    if (lane == 0) umma::mbar_expect_tx(umma::smem_u32(&sh.bar[2]), CL * 8);
    if (lane < CL)
      send2(umma::map_to_rank(umma::smem_u32(&sh.minmax[rank][0]), lane), umma::map_to_rank(umma::smem_u32(&sh.bar[2]), lane),
            kmin, kmax);
    inbox_wait(sh, 2, 0, status);
    kmin = sh.minmax[lane & (CL - 1)][0]; kmax = sh.minmax[lane & (CL - 1)][1];
#pragma unroll
    for (int o = CL / 2; o > 0; o >>= 1) {
      kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
      kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
    }
    const unsigned diff = kmin ^ kmax;
    const int nbits = diff ? 32 - __clz(diff) : 0;
    if (lane == 0) {
      sh.prefix = nbits >= 32 ? 0u : kmin & ~((1u << nbits) - 1u);
      sh.remaining = K;
      sh.sure = 0;
      sh.warp_tot[NW] = nbits;
    }
  }
  __syncthreads();
  return sh.warp_tot[NW];
}

// After the histograms of one pass are filled: sum them per CTA, send the sums to every CTA of the
// cluster, add up the eight that arrive here and narrow (prefix, remaining) by one digit; leaves the
// histograms zeroed.  The inbox
// written in pass p was last read in pass p - 2, and a CTA can only be two passes ahead of another
// after that one has sent its pass p - 1 histogram, i.e. after it finished reading pass p - 2.
__device__ __forceinline__ void cluster_select_digit(TopkShared& sh, int rank, int pass, int shift, uint32_t* status) {
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int buf = pass & 1;
  __syncthreads();
  if (tid < 256) {
    int s = 0;
#pragma unroll
    for (int w2 = 0; w2 < NH; ++w2) s += sh.hist[w2][tid];
    sh.cta_bins[tid] = s;
  }
  if (tid == 0) umma::mbar_expect_tx(umma::smem_u32(&sh.bar[buf]), CL * 256 * 4);
  __syncthreads();
  if (tid < CL * 64) {                               // 64 16-byte pieces to each of the eight CTAs
    const int to = tid >> 6, piece = tid & 63;
    const int4 v = reinterpret_cast<const int4*>(sh.cta_bins)[piece];
    send4(umma::map_to_rank(umma::smem_u32(&sh.inbox[buf][rank][4 * piece]), to),
          umma::map_to_rank(umma::smem_u32(&sh.bar[buf]), to), v);
  }
  hist_clear(sh);                                    // for the next pass, while the messages are under way
  if (wid == 0) {
    inbox_wait(sh, buf, (pass >> 1) & 1, status);
    // lane l owns bins 255-8l .. 248-8l (descending)
    const int remaining = sh.remaining;
    int loc[8], csum = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) loc[i] = 0;
#pragma unroll
    for (int rr = 0; rr < CL; ++rr) {
      const int4 hi4 = *reinterpret_cast<const int4*>(&sh.inbox[buf][rr][252 - 8 * lane]);
      const int4 lo4 = *reinterpret_cast<const int4*>(&sh.inbox[buf][rr][248 - 8 * lane]);
      loc[0] += hi4.w; loc[1] += hi4.z; loc[2] += hi4.y; loc[3] += hi4.x;
      loc[4] += lo4.w; loc[5] += lo4.z; loc[6] += lo4.y; loc[7] += lo4.x;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) csum += loc[i];
    int inc = csum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += n;
    }
    int excl = inc - csum;
    if (excl < remaining && remaining <= inc) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (excl + loc[i] >= remaining) {
          sh.prefix |= (unsigned)(255 - 8 * lane - i) << shift;
          sh.remaining = remaining - excl;
          sh.digit = 255 - 8 * lane - i;
          sh.alive = loc[i];
          break;
        }
        excl += loc[i];
      }
    }
  }
  __syncthreads();
}

// Short-cut once few keys are left: when at most LIST_CAP keys of the whole cluster still match the prefix
// after a pass (typically a dozen after two passes), every CTA sends its matching keys to all CTAs -- the
// per-CTA counts, hence every key's place on the list and the number of bytes to wait for, are in the
// histograms that were just exchanged -- and each CTA finds the wanted key among them by counting, instead
// of one more exchange per remaining digit.  Sets (prefix, remaining) to the final (threshold key, number
// of keys equal to it that are taken).
template <bool FULL>
__device__ __forceinline__ void list_send(TopkShared& sh, const unsigned (&keys)[16], int nmine, unsigned mask,
                                          unsigned prefix, int my_off) {
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    if ((FULL || k < nmine) && (keys[k] & mask) == prefix) {
      const int slot = my_off + atomicAdd(&sh.list_n, 1);
      if (slot < LIST_CAP) {
        const uint32_t dst = umma::smem_u32(&sh.list[slot]), bar = umma::smem_u32(&sh.bar[4]);
        for (int to = 0; to < CL; ++to) send1(umma::map_to_rank(dst, to), umma::map_to_rank(bar, to), keys[k]);
      }
    }
  }
}
__device__ __forceinline__ int list_offset(const TopkShared& sh, int rank, int buf) {
  int off = 0;
  const int digit = sh.digit;
#pragma unroll
  for (int rr = 0; rr < CL; ++rr) off += rr < rank ? sh.inbox[buf][rr][digit] : 0;   // independent loads
  return off;
}
__device__ __forceinline__ void list_finish(TopkShared& sh, uint32_t* status) {
  const int tid = threadIdx.x, n = sh.alive, want = sh.remaining;
  if (tid == 0) umma::mbar_expect_tx(umma::smem_u32(&sh.bar[4]), n * 4);
  const int i = tid >> 2, part = tid & 3;            // four threads count for key i, a quarter of the list each
  if (tid < ((4 * n + 31) & ~31)) inbox_wait(sh, 4, 0, status);   // the warps that hold a key
  __syncthreads();                                   // everyone has read `want` before it is overwritten
  if (tid < ((4 * n + 31) & ~31)) {
    const unsigned mine = sh.list[min(i, n - 1)];
    int g = 0, e = 0;
    for (int j = 4 * part; j < n; j += 16) {
      const uint4 o = *reinterpret_cast<const uint4*>(&sh.list[j]);
      g += (o.x > mine) + (j + 1 < n && o.y > mine) + (j + 2 < n && o.z > mine) + (j + 3 < n && o.w > mine);
      e += (o.x == mine) + (j + 1 < n && o.y == mine) + (j + 2 < n && o.z == mine) + (j + 3 < n && o.w == mine);
    }
    g += __shfl_xor_sync(0xffffffffu, g, 1); e += __shfl_xor_sync(0xffffffffu, e, 1);
    g += __shfl_xor_sync(0xffffffffu, g, 2); e += __shfl_xor_sync(0xffffffffu, e, 2);
    if (i < n && part == 0 && g < want && want <= g + e) { sh.prefix = mine; sh.remaining = want - g; }   // equal keys write the same
  }
  __syncthreads();
}

// Output offsets of this CTA's slice from the per-CTA (greater, equal) counts of the lower ranks.
__device__ __forceinline__ void cluster_offsets(TopkShared& sh, int rank, int tot_gt, int tot_eq, int need_eq,
                                                int& run_eq, int& run_out, uint32_t* status) {
  const int tid = threadIdx.x;
  if (tid == 0) umma::mbar_expect_tx(umma::smem_u32(&sh.bar[3]), CL * 8);
  if (tid < CL)
    send2(umma::map_to_rank(umma::smem_u32(&sh.counts[rank][0]), tid), umma::map_to_rank(umma::smem_u32(&sh.bar[3]), tid),
          (unsigned)tot_gt, (unsigned)tot_eq);
  inbox_wait(sh, 3, 0, status);
  run_eq = 0; run_out = 0;
  for (int rr = 0; rr < rank; ++rr) {
    const int g = sh.counts[rr][0], e = sh.counts[rr][1];
    run_out += g + min(max(need_eq - run_eq, 0), e);
    run_eq += e;
  }
}

__device__ __forceinline__ bool trivial_case(const TopkArgs& a, int seq, int Le, int rank, int* out) {
  if (Le > a.K && a.b.score_idx[seq] >= 0) return false;
  const int nv = max(min(Le, a.K), 0);               // keep every candidate (or none); whole cluster
  for (int i = rank * NT + threadIdx.x; i < a.K; i += CL * NT) out[i] = i < nv ? a.Ls + i : -1;
  return true;
}

// Emission of one thread's keys (register-resident kernel).  One pass over the sixteen keys builds three
// bit masks (above the threshold, equal to it, inside the re-scoring band); everything after that walks set
// bits only -- a thread selects half a key on average and band members are a handful per head -- so the
// per-key cost is three comparisons instead of a predicated store, a branch and an atomic's worth of code
// per key (this step took 5.5 us of the kernel's 20 us on a 128k-token prompt, 0.8 us now).
struct KeyMasks { unsigned gt, eq, band; };
template <bool FULL>
__device__ __forceinline__ KeyMasks classify_keys(const unsigned (&keys)[16], int nmine, unsigned tau, unsigned band_lo,
                                                  unsigned band_span) {
  KeyMasks m = {0u, 0u, 0u};
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    if (FULL || k < nmine) {
      m.gt |= keys[k] > tau ? 1u << k : 0u;
      m.eq |= keys[k] == tau ? 1u << k : 0u;
      m.band |= keys[k] - band_lo <= band_span ? 1u << k : 0u;
    }
  }
  return m;
}
__device__ __forceinline__ unsigned key_at(const unsigned (&keys)[16], int k) {   // rare paths only
  unsigned v = 0u;
#pragma unroll
  for (int kk = 0; kk < 16; ++kk) v = kk == k ? keys[kk] : v;
  return v;
}
// Writes the selected positions (ascending) from out[pos] on and records the band members; returns how many
// of the thread's keys lie above the band.  eq_take: how many of the thread's threshold-equal keys are taken
// (the first ones in index order).
__device__ __forceinline__ int emit_keys(const TopkArgs& a, const Band& bd, const unsigned (&keys)[16], KeyMasks m,
                                         int eq_take, int pos, int base, int* out) {
  unsigned sel = m.gt, eq = m.eq;
  for (; eq_take > 0 && eq; --eq_take) { sel |= eq & (0u - eq); eq &= eq - 1u; }
  const int val0 = a.Ls + base;
  for (unsigned left = sel; left; left &= left - 1u, ++pos)
    if (index_ok(pos, a.K, a.status)) out[pos] = val0 + (__ffs((int)left) - 1);
  int above_in_band = 0;
  for (unsigned left = m.band; left; left &= left - 1u) {
    const int k = __ffs((int)left) - 1;
    band_record(bd, key_at(keys, k), base + k, (sel >> k) & 1u);
    above_in_band += (m.gt >> k) & 1u;
  }
  return __popc(m.gt) - above_in_band;               // keys above the threshold that are not in the band
}

// ---- register-resident kernel: thread t of rank r owns candidates [j0 + 16t, j0 + 16t + 16) ----
// R = half the pooling width when it is known at compile time (the paper's width 7 -> 3), -1 = any width up
// to 2 * MAXR + 1.  Slices start on multiples of four candidates so that a thread fetches its window
// [base - 8, base + 24) as eight aligned 16-byte loads (thirty-two scalar loads took 7 of the kernel's 21 us
// on a 128k-token prompt).
template <int R>
__global__ void __cluster_dims__(CL, 1, 1) __launch_bounds__(NT) pool_topk_regs_kernel(const TopkArgs a) {
  pdl_wait();
  __shared__ TopkShared sh;
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int seq = blockIdx.z, kvh = blockIdx.y;
  const int Le = a.b.len[seq] - a.Ls - a.Lr;
  int* out = a.idx_out + ((long long)(a.b.first_seq + seq) * a.Hkv + kvh) * a.K;
  const int tid = threadIdx.x, wid = tid >> 5;
  if (trivial_case(a, seq, Le, rank, out)) return;

  const long long z = (long long)a.b.score_idx[seq] * a.Hkv + kvh;
  band_reset(a, z, rank);
  inbox_init(sh);
  cluster.barrier_arrive();                          // completed in cluster_common_prefix
  hist_clear(sh);
  const float* __restrict__ C = a.buf.C + z * a.buf.c_stride;    // 16-byte aligned rows of c_stride (a multiple of 64) floats
  const int j0 = rank == 0 ? 0 : (int)((long long)Le * rank / CL) & ~3;
  const int j1 = rank == CL - 1 ? Le : (int)((long long)Le * (rank + 1) / CL) & ~3;
  const int base = j0 + tid * MAXE;                  // first candidate of this thread
  const int nmine = max(0, min(MAXE, j1 - base));
  // Warp-uniform choices: a warp runs one variant of each loop (the slice's last partly filled warp would
  // otherwise run two, and every barrier waits for it).
  const bool warp_full = __all_sync(0xffffffffu, nmine == MAXE), warp_some = __any_sync(0xffffffffu, nmine > 0);

  // ---- load the score window once and pool it in registers: win[i] is candidate base - MAXR + i ----
  const int r = R >= 0 ? R : a.w / 2;
  const bool avg = a.pool_mode == SNAP_POOL_AVG;
  const float pad = avg ? 0.f : -INFINITY, inv_w = 1.0f / (float)a.w;
  unsigned keys[MAXE];
  if (warp_some) {                                   // whole warps past the end of a short slice skip this
    float win[MAXE + 2 * MAXR];
#pragma unroll
    for (int c = 0; c < (MAXE + 2 * MAXR) / 4; ++c) {
      const int jj = base - MAXR + 4 * c;            // a multiple of four: the piece lies inside the row or outside it
      float4 v = make_float4(pad, pad, pad, pad);
      if (nmine > 0 && jj >= 0 && jj < Le) v = *reinterpret_cast<const float4*>(C + jj);
      win[4 * c + 0] = v.x;
      win[4 * c + 1] = jj + 1 < Le ? v.y : pad;
      win[4 * c + 2] = jj + 2 < Le ? v.z : pad;
      win[4 * c + 3] = jj + 3 < Le ? v.w : pad;
    }
#pragma unroll
    for (int k = 0; k < MAXE; ++k) {
      float s = pad;
      if (R >= 0) {
#pragma unroll
        for (int t = MAXR - R; t <= MAXR + R; ++t) s = avg ? s + win[k + t] : fmaxf(s, win[k + t]);
      } else {
#pragma unroll
        for (int t = 0; t < 2 * MAXR + 1; ++t)
          if (t >= MAXR - r && t <= MAXR + r) s = avg ? s + win[k + t] : fmaxf(s, win[k + t]);
      }
      keys[k] = key_of(avg ? s * inv_w : s);
    }
  } else {
#pragma unroll
    for (int k = 0; k < MAXE; ++k) keys[k] = 0u;
  }
  // ---- radix select of the K-th largest key over the whole cluster ----
  unsigned kmin = 0xffffffffu, kmax = 0u;
#pragma unroll
  for (int k = 0; k < MAXE; ++k)
    if (k < nmine) { kmin = min(kmin, keys[k]); kmax = max(kmax, keys[k]); }
  const int nbits = cluster_common_prefix(cluster, sh, rank, kmin, kmax, a.K, a.status);
  unsigned mask = nbits >= 32 ? 0u : ~((1u << nbits) - 1u);
  int pass = 0;
  for (int hi = nbits - 1; hi >= 0; hi -= 8, ++pass) {
    const int shift = max(hi - 7, 0);
    const unsigned dmask = (1u << (hi - shift + 1)) - 1u;
    const unsigned prefix = sh.prefix;
    if (warp_full) hist_keys<true>(sh.hist[wid >> 1], keys, nmine, mask, prefix, shift, dmask);
    else if (warp_some) hist_keys<false>(sh.hist[wid >> 1], keys, nmine, mask, prefix, shift, dmask);
    cluster_select_digit(sh, rank, pass, shift, a.status);
    mask |= dmask << shift;
    if (shift > 0 && sh.alive > 0 && sh.alive <= LIST_CAP) {         // the same decision in every CTA of the cluster
      const int my_off = list_offset(sh, rank, pass & 1);
      if (warp_full) list_send<true>(sh, keys, nmine, mask, sh.prefix, my_off);
      else if (warp_some) list_send<false>(sh, keys, nmine, mask, sh.prefix, my_off);
      list_finish(sh, a.status);
      break;
    }
  }
  const unsigned tau = sh.prefix;      // key of the K-th largest pooled score
  const int need_eq = sh.remaining;    // how many keys equal to tau are taken (>= 1)

  // ---- ordered emission: thread order is index order, so one scan places everything.  The scan carries
  // (greater, equal) counts in the two halves of one word (at most 16384 each per CTA); equal keys are taken
  // in index order until the quota is used up, so of the e equal keys before a thread min(e, quota) were taken.
  const Band bd = make_band(a, z, tau);
  const unsigned band_lo = bd.head ? bd.lo : 1u, band_span = bd.head ? bd.hi - bd.lo : 0u;
  KeyMasks m = {0u, 0u, 0u};
  if (warp_full) m = classify_keys<true>(keys, nmine, tau, band_lo, band_span);
  else if (warp_some) m = classify_keys<false>(keys, nmine, tau, band_lo, band_span);
  if (!bd.head) m.band = 0u;
  const int gt_t = __popc(m.gt), eq_t = __popc(m.eq);
  int tot_pair;
  const int before = block_exscan((gt_t << 16) | eq_t, sh.warp_tot, tot_pair);
  const int eq_before = before & 0xffff, gt_before = before >> 16;
  int run_eq, run_out;
  cluster_offsets(sh, rank, tot_pair >> 16, tot_pair & 0xffff, need_eq, run_eq, run_out, a.status);
  __syncthreads();
  if (sh.failed) return;
  const int quota = max(need_eq - run_eq, 0);        // equal keys this CTA may still take
  const int pos = run_out + gt_before + min(eq_before, quota);
  int sure = 0;
  if (m.gt | m.eq | m.band) sure = emit_keys(a, bd, keys, m, min(max(quota - eq_before, 0), eq_t), pos, base, out);
  if (bd.head) band_count_sure(bd, sure, &sh.sure);
}

// ---- streaming kernel: any length and pooling width; pooled scores live in scratch ----
__global__ void __cluster_dims__(CL, 1, 1) __launch_bounds__(NT) pool_topk_stream_kernel(const TopkArgs a) {
  pdl_wait();
  __shared__ TopkShared sh;
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int seq = blockIdx.z, kvh = blockIdx.y;
  const int Le = a.b.len[seq] - a.Ls - a.Lr;
  int* out = a.idx_out + ((long long)(a.b.first_seq + seq) * a.Hkv + kvh) * a.K;
  const int tid = threadIdx.x, wid = tid >> 5;
  if (trivial_case(a, seq, Le, rank, out)) return;

  const long long z = (long long)a.b.score_idx[seq] * a.Hkv + kvh;
  band_reset(a, z, rank);
  inbox_init(sh);
  cluster.barrier_arrive();                          // completed in cluster_common_prefix
  hist_clear(sh);
  const long long zoff = z * a.buf.c_stride;
  const float* __restrict__ C = a.buf.C + zoff;
  float* __restrict__ P = a.buf.P + zoff;
  const int j0 = (int)((long long)Le * rank / CL), j1 = (int)((long long)Le * (rank + 1) / CL);

  const int r = a.w / 2;
  const bool avg = a.pool_mode == SNAP_POOL_AVG;
  const float inv_w = 1.0f / (float)a.w;
  for (int j = j0 + tid; j < j1; j += NT) {
    float s = avg ? 0.f : -INFINITY;
    for (int t = -r; t <= r; ++t) {
      const int jj = j + t;
      if (jj >= 0 && jj < Le) s = avg ? s + C[jj] : fmaxf(s, C[jj]);
    }
    P[j] = avg ? s * inv_w : s;
  }
  __syncthreads();
  unsigned kmin = 0xffffffffu, kmax = 0u;
  for (int j = j0 + tid; j < j1; j += NT) {          // a thread re-reads only what it wrote itself
    const unsigned key = key_of(P[j]);
    kmin = min(kmin, key); kmax = max(kmax, key);
  }
  const int nbits = cluster_common_prefix(cluster, sh, rank, kmin, kmax, a.K, a.status);
  unsigned mask = nbits >= 32 ? 0u : ~((1u << nbits) - 1u);
  int pass = 0;
  for (int hi = nbits - 1; hi >= 0; hi -= 8, ++pass) {
    const int shift = max(hi - 7, 0);
    const unsigned dmask = (1u << (hi - shift + 1)) - 1u;
    const unsigned prefix = sh.prefix;
    for (int j = j0 + tid; j < j1; j += NT)
      hist_add(sh.hist[wid >> 1], key_of(P[j]), mask, prefix, shift, dmask);
    cluster_select_digit(sh, rank, pass, shift, a.status);
    mask |= dmask << shift;
  }
  const unsigned tau = sh.prefix;
  const int need_eq = sh.remaining;

  int my_gt = 0, my_eq = 0, tot_gt, tot_eq;
  for (int j = j0 + tid; j < j1; j += NT) {
    const unsigned key = key_of(P[j]);
    my_gt += key > tau;
    my_eq += key == tau;
  }
  (void)block_exscan(my_gt, sh.warp_tot, tot_gt);
  (void)block_exscan(my_eq, sh.warp_tot, tot_eq);
  int run_eq, run_out;
  cluster_offsets(sh, rank, tot_gt, tot_eq, need_eq, run_eq, run_out, a.status);
  __syncthreads();
  if (sh.failed) return;

  const Band bd = make_band(a, z, tau);
  int sure = 0;
  for (int tb = j0; tb < j1; tb += NT) {             // ordered emission, 1024 candidates at a time
    const int j = tb + tid;
    const unsigned key = j < j1 ? key_of(P[j]) : 0u;
    const bool gt = j < j1 && key > tau;
    const bool eq = j < j1 && key == tau;
    int te, ts;
    const int rank_eq = block_exscan(eq, sh.warp_tot, te);
    const bool sel = gt || (eq && run_eq + rank_eq < need_eq);
    const int rank_sel = block_exscan(sel, sh.warp_tot, ts);
    if (sel && index_ok(run_out + rank_sel, a.K, a.status)) out[run_out + rank_sel] = a.Ls + j;
    if (bd.head && j < j1) {
      band_record(bd, key, j, sel);
      sure += key > bd.hi;
    }
    run_eq += te;
    run_out += ts;
  }
  if (bd.head) band_count_sure(bd, sure, &sh.sure);
}

}  // namespace

cudaError_t launch_pool_topk(const Shape& s, const SeqBatch& b, const ScoreBuffers& buf,
                             int* idx_out, uint32_t* status, cudaStream_t st) {
  if (s.K == 0 || b.n == 0) return cudaSuccess;
  TopkArgs a;
  a.Hkv = s.Hkv; a.Ls = s.Ls; a.Lr = s.Lr; a.K = s.K; a.w = s.w; a.pool_mode = s.pool_mode;
  a.b = b; a.buf = buf; a.idx_out = idx_out; a.status = status;
  int max_le = 0;
  for (int i = 0; i < b.n; ++i) max_le = max(max_le, b.len[i] - s.Ls - s.Lr);
  dim3 grid(CL, s.Hkv, b.n);
  cudaError_t e;
  if ((max_le + CL - 1) / CL + 4 <= MAXE * NT && s.w / 2 <= MAXR)        // slices are cut at multiples of four
    e = s.w / 2 == 3 ? launch_pdl(pool_topk_regs_kernel<3>, grid, dim3(NT), 0, st, a)
                     : launch_pdl(pool_topk_regs_kernel<-1>, grid, dim3(NT), 0, st, a);
  else
    e = launch_pdl(pool_topk_stream_kernel, grid, dim3(NT), 0, st, a);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace snap
