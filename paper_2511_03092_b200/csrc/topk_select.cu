// Sequence-axis pooling and per-KV-head top-K (Eq. 2), one cluster of 8 CTAs per (prompt, KV head).
//
//   P[j] = pool_w(C)[j]  (1-D, stride 1, pad w/2; average divides by w over zero padding, max pads -inf)
//   keep the K largest P, ties to the lower index, and emit absolute positions in ascending order.
//
// Each CTA of the cluster owns a contiguous eighth of the candidates.  Selection is an
// 8-bit-digit radix select on the order-preserving integer image of P: four histogram passes
// narrow down the K-th largest key (the high bits that all keys share are found first with a
// cluster-wide min/max and skipped).  Histograms are per warp in shared memory, summed per CTA,
// and every CTA adds up the eight CTA
// histograms through distributed shared memory, so all of them find the same digit without a
// broadcast.  Then an ordered compaction: every key above the threshold is taken, and of the
// keys equal to it the first ones in index order until K are reached; CTA offsets come from the
// per-CTA counts (again exchanged through DSMEM) -- no global atomics, deterministic output.
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

namespace cg = cooperative_groups;

namespace snap {
namespace {

constexpr int NT = 1024, NW = NT / 32, CL = 8, MAXE = 16, MAXR = 8;

struct TopkArgs {
  int Hkv, Ls, Lr, K, w, pool_mode;
  SeqBatch b;
  ScoreBuffers buf;
  int* idx_out;      // [n][Hkv][K]
  uint32_t* status;
};

struct TopkShared {
  int hist[NW][256];
  int bins[2][256];      // this CTA's histogram (double buffered), read by the whole cluster
  int counts[2];         // this CTA's (greater, equal) counts, read by the whole cluster
  int warp_tot[NW + 1];
  int tot[256];          // cluster-wide histogram of the current pass
  unsigned prefix;
  int remaining;
  int sure;              // this CTA's candidates above the re-scoring band
};

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

// One histogram update (per-warp histogram, shared-memory atomic).
__device__ __forceinline__ void hist_add(int* warp_hist, unsigned key, unsigned mask, unsigned prefix, int shift,
                                         unsigned dmask) {
  if ((key & mask) == prefix) atomicAdd(&warp_hist[(key >> shift) & dmask], 1);
}

// Smallest and largest key of the cluster.  The bits above the highest bit in which they differ
// are common to every key and need no histogram pass (pooled scores share sign and most of the
// exponent, so the leading digit would otherwise put a whole warp on one counter).
// Returns the number of low bits still to be resolved; sets sh.prefix to the common high bits.
__device__ __forceinline__ int cluster_common_prefix(cg::cluster_group& cluster, TopkShared& sh, unsigned kmin,
                                                     unsigned kmax, int K) {
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
    kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
  }
  unsigned* mm = reinterpret_cast<unsigned*>(&sh.hist[0][0]);       // [0..31] warp minima, [32..63] maxima
  if (lane == 0) { mm[wid] = kmin; mm[32 + wid] = kmax; }
  __syncthreads();
  if (wid == 0) {
    kmin = mm[lane]; kmax = mm[32 + lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
      kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
    }
    if (lane == 0) { sh.bins[0][0] = (int)kmin; sh.bins[0][1] = (int)kmax; }
  }
  cluster.sync();
  kmin = 0xffffffffu; kmax = 0u;
  for (int rr = 0; rr < CL; ++rr) {
    const int* rb = cluster.map_shared_rank(sh.bins[0], rr);
    kmin = min(kmin, (unsigned)rb[0]);
    kmax = max(kmax, (unsigned)rb[1]);
  }
  cluster.sync();                                    // bins[0] is reused by the first histogram pass
  const unsigned diff = kmin ^ kmax;
  const int nbits = diff ? 32 - __clz(diff) : 0;
  if (tid == 0) {
    sh.prefix = nbits >= 32 ? 0u : kmin & ~((1u << nbits) - 1u);
    sh.remaining = K;
    sh.sure = 0;
  }
  __syncthreads();
  return nbits;
}

// After the per-warp histograms of one pass are filled: sum them per CTA, add up the cluster's
// CTAs through DSMEM and narrow (prefix, remaining) by one digit.  One cluster barrier per pass:
// the bins buffer written now was last read two passes ago, with a barrier in between.
__device__ __forceinline__ void cluster_select_digit(cg::cluster_group& cluster, TopkShared& sh, int pass, int shift) {
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  __syncthreads();
  int* mybins = sh.bins[pass & 1];
  if (tid < 256) {
    int s = 0;
#pragma unroll 8
    for (int w2 = 0; w2 < NW; ++w2) s += sh.hist[w2][tid];
    mybins[tid] = s;
  }
  cluster.sync();
  if (tid < 256) {                                   // one bin per thread, eight independent remote reads
    int s = 0;
#pragma unroll
    for (int rr = 0; rr < CL; ++rr) s += cluster.map_shared_rank(mybins, rr)[tid];
    sh.tot[tid] = s;
  }
  __syncthreads();
  if (wid == 0) {
    // lane l owns bins 255-8l .. 248-8l (descending)
    const int remaining = sh.remaining;
    int loc[8], csum = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) loc[i] = sh.tot[255 - 8 * lane - i];
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
          break;
        }
        excl += loc[i];
      }
    }
  }
  __syncthreads();
}

// Output offsets of this CTA's slice from the per-CTA (greater, equal) counts of the lower ranks.
__device__ __forceinline__ void cluster_offsets(cg::cluster_group& cluster, TopkShared& sh, int rank, int need_eq,
                                                int& run_eq, int& run_out) {
  cluster.sync();
  run_eq = 0; run_out = 0;
  for (int rr = 0; rr < rank; ++rr) {
    const int* rc = cluster.map_shared_rank(sh.counts, rr);
    const int g = rc[0], e = rc[1];
    run_out += g + min(max(need_eq - run_eq, 0), e);
    run_eq += e;
  }
  cluster.sync();                                    // nobody leaves while its shared memory may still be read
}

__device__ __forceinline__ bool trivial_case(const TopkArgs& a, int seq, int Le, int rank, int* out) {
  if (Le > a.K && a.b.score_idx[seq] >= 0) return false;
  const int nv = max(min(Le, a.K), 0);               // keep every candidate (or none); whole cluster
  for (int i = rank * NT + threadIdx.x; i < a.K; i += CL * NT) out[i] = i < nv ? a.Ls + i : -1;
  return true;
}

// ---- register-resident kernel: thread t of rank r owns candidates [j0 + 16t, j0 + 16t + 16) ----
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
  const float* __restrict__ C = a.buf.C + z * a.buf.c_stride;
  const int j0 = (int)((long long)Le * rank / CL), j1 = (int)((long long)Le * (rank + 1) / CL);
  const int base = j0 + tid * MAXE;                  // first candidate of this thread
  const int nmine = max(0, min(MAXE, j1 - base));

  // ---- load the score window once and pool it in registers ----
  const int r = a.w / 2;
  const bool avg = a.pool_mode == SNAP_POOL_AVG;
  const float pad = avg ? 0.f : -INFINITY, inv_w = 1.0f / (float)a.w;
  float win[MAXE + 2 * MAXR];
#pragma unroll
  for (int i = 0; i < MAXE + 2 * MAXR; ++i) {
    const int jj = base - r + i;
    win[i] = (nmine > 0 && i < MAXE + 2 * r && jj >= 0 && jj < Le) ? C[jj] : pad;
  }
  unsigned keys[MAXE];
#pragma unroll
  for (int k = 0; k < MAXE; ++k) {
    float s = pad;
#pragma unroll
    for (int t = 0; t < 2 * MAXR + 1; ++t)
      if (t <= 2 * r) s = avg ? s + win[k + t] : fmaxf(s, win[k + t]);
    keys[k] = key_of(avg ? s * inv_w : s);
  }
  // ---- radix select of the K-th largest key over the whole cluster ----
  unsigned kmin = 0xffffffffu, kmax = 0u;
#pragma unroll
  for (int k = 0; k < MAXE; ++k)
    if (k < nmine) { kmin = min(kmin, keys[k]); kmax = max(kmax, keys[k]); }
  const int nbits = cluster_common_prefix(cluster, sh, kmin, kmax, a.K);
  unsigned mask = nbits >= 32 ? 0u : ~((1u << nbits) - 1u);
  int pass = 0;
  for (int hi = nbits - 1; hi >= 0; hi -= 8, ++pass) {
    const int shift = max(hi - 7, 0);
    const unsigned dmask = (1u << (hi - shift + 1)) - 1u;
    for (int i = tid; i < NW * 256; i += NT) (&sh.hist[0][0])[i] = 0;
    __syncthreads();
    const unsigned prefix = sh.prefix;
#pragma unroll
    for (int k = 0; k < MAXE; ++k)
      if (k < nmine) hist_add(sh.hist[wid], keys[k], mask, prefix, shift, dmask);
    cluster_select_digit(cluster, sh, pass, shift);
    mask |= dmask << shift;
  }
  const unsigned tau = sh.prefix;      // key of the K-th largest pooled score
  const int need_eq = sh.remaining;    // how many keys equal to tau are taken (>= 1)

  // ---- ordered emission: thread order is index order, so one scan places everything ----
  int gt_t = 0, eq_t = 0;
#pragma unroll
  for (int k = 0; k < MAXE; ++k) {
    gt_t += k < nmine && keys[k] > tau;
    eq_t += k < nmine && keys[k] == tau;
  }
  int tot_gt, tot_eq, tot_sel;
  const int eq_before = block_exscan(eq_t, sh.warp_tot, tot_eq);
  (void)block_exscan(gt_t, sh.warp_tot, tot_gt);
  if (tid == 0) { sh.counts[0] = tot_gt; sh.counts[1] = tot_eq; }
  int run_eq, run_out;
  cluster_offsets(cluster, sh, rank, need_eq, run_eq, run_out);
  int eq_left = min(max(need_eq - (run_eq + eq_before), 0), eq_t);
  int pos = run_out + block_exscan(gt_t + eq_left, sh.warp_tot, tot_sel);
  const Band bd = make_band(a, z, tau);
  int sure = 0;
#pragma unroll
  for (int k = 0; k < MAXE; ++k) {
    if (k < nmine) {
      bool sel = keys[k] > tau;
      if (keys[k] == tau && eq_left > 0) { sel = true; --eq_left; }
      if (sel && index_ok(pos, a.K, a.status)) out[pos] = a.Ls + base + k;
      pos += sel;
      if (bd.head) {
        band_record(bd, keys[k], base + k, sel);
        sure += keys[k] > bd.hi;
      }
    }
  }
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
  const int nbits = cluster_common_prefix(cluster, sh, kmin, kmax, a.K);
  unsigned mask = nbits >= 32 ? 0u : ~((1u << nbits) - 1u);
  int pass = 0;
  for (int hi = nbits - 1; hi >= 0; hi -= 8, ++pass) {
    const int shift = max(hi - 7, 0);
    const unsigned dmask = (1u << (hi - shift + 1)) - 1u;
    for (int i = tid; i < NW * 256; i += NT) (&sh.hist[0][0])[i] = 0;
    __syncthreads();
    const unsigned prefix = sh.prefix;
    for (int j = j0 + tid; j < j1; j += NT)
      hist_add(sh.hist[wid], key_of(P[j]), mask, prefix, shift, dmask);
    cluster_select_digit(cluster, sh, pass, shift);
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
  if (tid == 0) { sh.counts[0] = tot_gt; sh.counts[1] = tot_eq; }
  int run_eq, run_out;
  cluster_offsets(cluster, sh, rank, need_eq, run_eq, run_out);

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
  if ((max_le + CL - 1) / CL + 1 <= MAXE * NT && s.w / 2 <= MAXR)
    e = launch_pdl(pool_topk_regs_kernel, grid, dim3(NT), 0, st, a);
  else
    e = launch_pdl(pool_topk_stream_kernel, grid, dim3(NT), 0, st, a);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace snap
