// Decode attention over the compressed cache for the latent-attention layout (Section 3.3 with
// the paper's remark that the latent vectors are what gets compressed): one KV "head" whose row
// is 512 latent dims followed by 64 rotary dims, scores on all 576 dims, values = the 512 latent
// dims of the same row, and many query heads (128) sharing that row.
//
// With 128 heads per row this is a real contraction (about 240 flop per cache byte), so both
// products run on the tensor cores (mma.sync.m16n8k16, bf16 in, fp32 accumulate).
// Grid = (splits, blocks of 64 heads, sequences), 8 warps per CTA: warp (t, h) owns the 16 heads
// of head tile t and half h of the 512 output dims, so its output accumulator is 16 x 256 fp32
// (128 registers).  The query block (64 x 576) stays in shared memory; cache rows stream through
// a 3-stage cp.async ring of 32-row tiles in an XOR-swizzled layout (conflict-free ldmatrix);
// the same staged tile is the B operand of Q.K^T (plain ldmatrix) and of P.V (ldmatrix.trans).
// Logits stay in registers: the accumulator fragments of Q.K^T are exponentiated and repacked as
// the A fragments of P.V.  Online softmax per warp with a lazily refreshed reference max.
// The new token's row (Eq. 3) is substituted while staging and stored by the owning CTA.
#include "mma_helpers.cuh"
#include "snap_internal.cuh"

namespace snap {
namespace {

using namespace mmasync;

constexpr int DQK = 576, DV = 512, HB = 64, TR = 32, NSTG = 3, NT = 256;
constexpr int ROW_B = DQK * 2;                 // 1152 bytes per cache row
constexpr int CHUNKS = ROW_B / 16;             // 72 16-byte chunks per row
constexpr int QS_B = HB * ROW_B, KT_B = TR * ROW_B;
constexpr int PSM = DV + 4;                    // floats per partial: m, l, two unused, acc[DV] (rows 16-byte aligned)

struct MlaArgs {
  const __nv_bfloat16* q; const __nv_bfloat16* k_new;
  const int* slot_ids;
  char* kc;
  long long seq_b;
  int Hq, Ls, Lr, max_seqs, nsplit;
  float scale_log2;
  const int* seq_len; const int* valid_topk;
  float* partials;                             // [n_active][Hq][nsplit][PSM], maxima in the log2 domain
  uint32_t* status;
};

// row r, 16-byte chunk c of a 1152-byte-pitch tile; chunks are XOR-swizzled within groups of 8
__device__ __forceinline__ uint32_t swz(int r, int c) { return r * ROW_B + ((c ^ (r & 7)) << 4); }

__global__ void __launch_bounds__(NT, 1) decode_mla_kernel(const MlaArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  const uint32_t qs = smem_u32(smem), ks0 = qs + QS_B;

  const int sp = blockIdx.x, hb = blockIdx.y, i = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  const int mt = w & 3, dh = w >> 2;                       // head tile, output-dim half
  const int slot = a.slot_ids[i];
  const bool bad = slot < 0 || slot >= a.max_seqs;
  const int Lsr = a.Ls + a.Lr;
  int n_low = 0, n_valid = 0, new_slot = -1;
  if (!bad) {
    const int t = a.seq_len[slot];
    n_low = min(t + (a.k_new ? 1 : 0), Lsr);
    n_valid = n_low + a.valid_topk[slot];
    if (a.k_new) new_slot = ring_slot(t, a.Ls, a.Lr);
  } else if (tid == 0 && sp == 0 && hb == 0 && a.status) {
    atomicOr(a.status, SNAP_DEV_BAD_SLOT);
  }
  const int ntiles = (n_valid + TR - 1) / TR;
  const int t_begin = (int)((long long)ntiles * sp / a.nsplit);
  const int t_end = (int)((long long)ntiles * (sp + 1) / a.nsplit);
  const int v1 = min(n_valid, t_end * TR);
  const int T = t_end - t_begin;
  char* kc = a.kc + slot * a.seq_b;
  const char* kn = reinterpret_cast<const char*>(a.k_new ? a.k_new + (long long)i * DQK : nullptr);

  // stage one 32-row tile: row index x < n_low is cache row x, the rest is row Lsr + (x - n_low);
  // the new token's slot is read from k_new; rows past the end are zero-filled
  auto load_tile = [&](int t, int stage) {
    const int va = (t_begin + t) * TR;
    const uint32_t dst = ks0 + stage * KT_B;
    for (int idx = tid; idx < TR * CHUNKS; idx += NT) {
      const int r = idx / CHUNKS, c = idx - r * CHUNKS;
      const int x = va + r;
      const bool ok = x < v1;
      const int cs = x < n_low ? x : Lsr + (x - n_low);
      const char* src = !ok ? kc : (cs == new_slot ? kn : kc + (long long)cs * ROW_B) + c * 16;
      cp_async16(dst + swz(r, c), src, ok ? 16u : 0u);
    }
  };

  if (T > 0) {
    const char* qb = reinterpret_cast<const char*>(a.q + ((long long)i * a.Hq + (long long)hb * HB) * DQK);
    for (int idx = tid; idx < HB * CHUNKS; idx += NT) {
      const int r = idx / CHUNKS, c = idx - r * CHUNKS;
      cp_async16(qs + swz(r, c), qb + (long long)r * ROW_B + c * 16, 16u);
    }
    load_tile(0, 0);
    cp_commit();
    if (T > 1) load_tile(1, 1);
    cp_commit();
  }
  // the CTA (head block 0) that owns the new token's slot stores it
  if (new_slot >= t_begin * TR && new_slot < v1 && hb == 0 && tid < CHUNKS)
    reinterpret_cast<uint4*>(kc + (long long)new_slot * ROW_B)[tid] = reinterpret_cast<const uint4*>(kn)[tid];

  float o[32][4];                                           // 16 heads x 256 dims: [n-tile][frag]
#pragma unroll
  for (int j = 0; j < 32; ++j)
#pragma unroll
    for (int f = 0; f < 4; ++f) o[j][f] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};   // rows lane/4 and lane/4 + 8

  // ldmatrix lane coordinates
  const int a_row = 16 * mt + (lane & 7) + ((lane >> 3) & 1) * 8, a_chk = lane >> 4;   // Q: + 2*ks
  const int b_row = (lane & 7) + (lane >> 4) * 8, b_chk = (lane >> 3) & 1;             // K rows as n: + 16*np, + 2*ks
  const int v_row = (lane & 7) + ((lane >> 3) & 1) * 8, v_chk = lane >> 4;             // V rows as k: + 16*kk, chunk + 2*np

  for (int t = 0; t < T; ++t) {
    const int stage = t % NSTG;
    if (t + 2 < T) load_tile(t + 2, (t + 2) % NSTG);
    cp_commit();
    cp_wait<2>();
    __syncthreads();
    const uint32_t kst = ks0 + stage * KT_B;

    // ---- S = Q K^T for 16 heads x 32 rows ----
    float s[4][4];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
      for (int f = 0; f < 4; ++f) s[nt][f] = 0.f;
#pragma unroll 4
    for (int ks = 0; ks < DQK / 16; ++ks) {
      uint32_t af[4], b0[4], b1[4];
      ldsm4(qs + swz(a_row, 2 * ks + a_chk), af);
      ldsm4(kst + swz(b_row, 2 * ks + b_chk), b0);
      ldsm4(kst + swz(b_row + 16, 2 * ks + b_chk), b1);
      mma16816(s[0], af, b0[0], b0[1]);
      mma16816(s[1], af, b0[2], b0[3]);
      mma16816(s[2], af, b1[0], b1[1]);
      mma16816(s[3], af, b1[2], b1[3]);
    }
    // thread holds rows (lane/4, lane/4+8) x cols 8nt + 2(lane%4) + {0,1}
    const int nrows = min(TR, v1 - (t_begin + t) * TR);
    float tmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
      for (int f = 0; f < 4; ++f) {
        const int col = 8 * nt + 2 * (lane & 3) + (f & 1);
        s[nt][f] = col < nrows ? s[nt][f] * a.scale_log2 : -INFINITY;
        tmax[f >> 1] = fmaxf(tmax[f >> 1], s[nt][f]);
      }
    // the reference max is refreshed only when some row of the warp sees a logit 8 above it
    const bool need = tmax[0] > m_run[0] + 8.f || tmax[1] > m_run[1] + 8.f;
    if (__any_sync(0xffffffffu, need)) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        float mx = tmax[h];
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float mn = fmaxf(m_run[h], mx);
        const float al = m_run[h] == -INFINITY ? 0.f : fast_exp2(m_run[h] - mn);
        m_run[h] = mn;
        l_run[h] *= al;
#pragma unroll
        for (int j = 0; j < 32; ++j) { o[j][2 * h] *= al; o[j][2 * h + 1] *= al; }
      }
    }
    // ---- P = exp2(S - m), repacked as A fragments (k = cache rows) ----
    uint32_t pa[2][4];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      float p[4];
#pragma unroll
      for (int f = 0; f < 4; ++f) {
        const float mref = m_run[f >> 1] == -INFINITY ? 0.f : m_run[f >> 1];
        p[f] = fast_exp2(s[nt][f] - mref);
        l_run[f >> 1] += p[f];
      }
      pa[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p[0], p[1]);
      pa[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p[2], p[3]);
    }
    // ---- O += P V over this warp's 256 output dims ----
#pragma unroll
    for (int kk = 0; kk < 2; ++kk) {
#pragma unroll
      for (int np = 0; np < 16; ++np) {
        uint32_t bv[4];
        ldsm4t(kst + swz(v_row + 16 * kk, dh * 32 + 2 * np + v_chk), bv);
        mma16816(o[2 * np], pa[kk], bv[0], bv[1]);
        mma16816(o[2 * np + 1], pa[kk], bv[2], bv[3]);
      }
    }
    __syncthreads();                                         // the stage is refilled two iterations later
  }
  cp_wait<0>();

  // ---- write the split's partial: (m, l) by the dh = 0 warp, its 256 dims by each warp ----
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 1);
    l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 2);
  }
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int head = hb * HB + 16 * mt + (lane >> 2) + 8 * h;
    float* ph = a.partials + (((long long)i * a.Hq + head) * a.nsplit + sp) * PSM;
    if (dh == 0 && (lane & 3) == 0) { ph[0] = m_run[h]; ph[1] = l_run[h]; }
#pragma unroll
    for (int j = 0; j < 32; ++j)
      *reinterpret_cast<float2*>(ph + 4 + dh * 256 + 8 * j + 2 * (lane & 3)) = make_float2(o[j][2 * h], o[j][2 * h + 1]);
  }
}

// Merge the splits of one (sequence, query head); maxima are in the log2 domain.  The split
// weights 2^(m_s - M) / L are computed once per block; a thread then sums four adjacent output
// dims over the splits with 16-byte loads.
__global__ void __launch_bounds__(128) decode_mla_merge_kernel(const float* __restrict__ partials,
                                                               __nv_bfloat16* __restrict__ out, int Hq, int nsplit,
                                                               const int* __restrict__ slot_ids, int* seq_len,
                                                               int max_seqs, int bump, int q_len, int u) {
  __shared__ float w_s[64];
  const int h = blockIdx.x, i = blockIdx.y;
  const float* p = partials + ((long long)i * Hq + h) * nsplit * PSM;
  // when launched as a programmatic dependent, wait for the split kernel's results (no-op otherwise)
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    float m0 = lane < nsplit ? p[lane * PSM] : -INFINITY, m1 = lane + 32 < nsplit ? p[(lane + 32) * PSM] : -INFINITY;
    float M = fmaxf(m0, m1);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    const float e0 = m0 != -INFINITY ? exp2f(m0 - M) : 0.f, e1 = m1 != -INFINITY ? exp2f(m1 - M) : 0.f;
    float L = (lane < nsplit ? p[lane * PSM + 1] * e0 : 0.f) + (lane + 32 < nsplit ? p[(lane + 32) * PSM + 1] * e1 : 0.f);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
    const float inv = L > 0.f ? 1.f / L : 0.f;
    w_s[lane] = e0 * inv;
    w_s[lane + 32] = e1 * inv;
  }
  __syncthreads();
  for (int dim = 4 * threadIdx.x; dim < DV; dim += 4 * blockDim.x) {
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < nsplit; ++s) {
      const float w = w_s[s];
      const float4 v = *reinterpret_cast<const float4*>(p + s * PSM + 4 + dim);
      o.x = fmaf(v.x, w, o.x); o.y = fmaf(v.y, w, o.y); o.z = fmaf(v.z, w, o.z); o.w = fmaf(v.w, w, o.w);
    }
    // out is [n_active][q_len][Hq][DV]: this launch serves token u of every sequence
    __nv_bfloat162* dst = reinterpret_cast<__nv_bfloat162*>(out + (((long long)i * q_len + u) * Hq + h) * DV + dim);
    dst[0] = __floats2bfloat162_rn(o.x, o.y);
    dst[1] = __floats2bfloat162_rn(o.z, o.w);
  }
  if (bump && h == 0 && threadIdx.x == 0) {
    const int slot = slot_ids[i];
    if (slot >= 0 && slot < max_seqs) seq_len[slot] += 1;
  }
}

}  // namespace

cudaError_t launch_decode_mla_merge(const float* partials, void* out, int n_active, int Hq, int nsplit,
                                    const int* slot_ids, int* seq_len, int max_seqs, int bump, cudaStream_t st,
                                    bool programmatic, int q_len, int u) {
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(Hq, (unsigned)n_active);
  lc.blockDim = dim3(128);
  lc.stream = st;
  lc.attrs = attr;
  lc.numAttrs = programmatic ? 1 : 0;
  cudaError_t e = cudaLaunchKernelEx(&lc, decode_mla_merge_kernel, partials, static_cast<__nv_bfloat16*>(out), Hq, nsplit,
                                     slot_ids, seq_len, max_seqs, bump, q_len, u);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

bool decode_mla_supported(int dtype, const Shape& s) {
  return dtype == SNAP_BF16 && s.v_aliases_k && s.d_qk == DQK && s.d_v == DV && s.Hkv == 1 && s.Hq % HB == 0;
}

// Splits per sequence: about one CTA per SM, at least two 32-row tiles per split.
int decode_mla_nsplit(const Shape& s, int n_active, int sm_count) {
  const int tiles = (s.Sc + TR - 1) / TR;
  const long long base = (long long)n_active * (s.Hq / HB);
  long long ns = (sm_count + base / 2) / base;
  if (ns > tiles / 2) ns = tiles / 2;
  if (ns > 64) ns = 64;
  if (ns < 1) ns = 1;
  return (int)ns;
}

size_t decode_mla_partial_floats(const Shape& s, int n_active, int nsplit) {
  return (size_t)n_active * s.Hq * nsplit * PSM;
}

cudaError_t launch_decode_mla(const Shape& s, const void* q, const void* k_new, const int* slot_ids,
                              int n_active, void* k_cache, int* seq_len, const int* valid_topk, void* out,
                              float* partials, int nsplit, uint32_t* status, cudaStream_t st) {
  if (n_active == 0) return cudaSuccess;
  MlaArgs a;
  a.q = static_cast<const __nv_bfloat16*>(q);
  a.k_new = static_cast<const __nv_bfloat16*>(k_new);
  a.slot_ids = slot_ids;
  a.kc = static_cast<char*>(k_cache);
  a.seq_b = (long long)s.Sc * ROW_B;
  a.Hq = s.Hq; a.Ls = s.Ls; a.Lr = s.Lr; a.max_seqs = s.max_seqs; a.nsplit = nsplit;
  a.scale_log2 = s.scale * 1.4426950408889634f;
  a.seq_len = seq_len; a.valid_topk = valid_topk; a.partials = partials; a.status = status;
  const size_t smem = QS_B + NSTG * KT_B;
  static SmemLimit limit = {};
  if (cudaError_t e = ensure_dyn_smem(decode_mla_kernel, smem, limit)) return e;
  dim3 grid(nsplit, s.Hq / HB, n_active);
  decode_mla_kernel<<<grid, NT, smem, st>>>(a);
  count_launch();
  dim3 mgrid(s.Hq, n_active);
  decode_mla_merge_kernel<<<mgrid, 128, 0, st>>>(partials, static_cast<__nv_bfloat16*>(out), s.Hq, nsplit,
                                                 slot_ids, seq_len, s.max_seqs, k_new != nullptr, 1, 0);
  count_launch();
  return cudaGetLastError();
}

}  // namespace snap
