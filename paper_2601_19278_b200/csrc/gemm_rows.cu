// Weight-streaming small-M GEMM for the draft layer's projections (FC, QKV, o_proj, gate/up,
// down -- Section 3.2's single decoder layer) with the op that follows each projection fused
// into its epilogue.
//
// The op is HBM-bound: M = batch*K token rows (8..128) against weight matrices of 10^7..10^8
// elements, i.e. M flop per weight byte.  The streaming loop is the shared core of
// stream_core.cuh (16 warps per CTA interleave k-steps over one 16-row tile; 2 CTAs per SM).
// What this file adds:
//   * stream-K: the flattened (16-row tile, k-round) space is cut into gridDim.x equal ranges, so
//     every CTA streams the same number of bytes (no tail wave).  A CTA writes one fp32 partial per
//     16-row tile it touches and takes tickets on the counter of the tile's 128-row group; the CTA
//     that takes the last ticket sums the group's partials in CTA order (deterministic, no float
//     atomics) and applies the fused op: residual add, RMSNorm gain + sum of squares, RoPE + cache
//     append, or SiLU-gate;
//   * RMSNorm's 1/rms is a per-token scalar, so it is applied *after* the next projection
//     (W (x*gain) * rstd): no row-wide reduction ever sits between two kernels.  A finalizer
//     only emits its group's partial sum of squares; whoever needs rstd adds up the groups'.
#include "common.cuh"
#include "kernels.h"
#include "stream_core.cuh"
#include "finalize.cuh"

namespace dart {

// Epilogue functor of the streaming core: partial write and tickets.  A CTA that takes the last ticket of
// a group only records the group; it runs the fused finalize after it has streamed its whole range, so the
// streaming loop stays free of the finalize's registers and latency.
template <int NT, int NW>
struct GemmEpi {
  static constexpr int MP = 8 * NT;
  const GemmArgs& p;
  const float* red;
  int* s_done;   // [0] = count, [1..] = completed groups
  int c, first_mt, pending;

  __device__ __forceinline__ int group_of(int mt) const {
    const int tile = mt >> 3;
    return p.pair_offset > 0 ? tile % p.pair_offset : tile;
  }
  __device__ __forceinline__ void after_wait() {}
  __device__ __forceinline__ void mtile_done(int mt, int buf, bool last) {
    float* dst = p.part + ((size_t)c * p.slots + (mt - first_mt)) * 16 * MP;
    for (int e = threadIdx.x; e < 16 * MP; e += blockDim.x) dst[e] = red_sum<NW, MP>(red, buf, e / MP, e % MP);
    ++pending;
    const int group = group_of(mt);
    if (last || group_of(mt + 1) != group) {
      // this CTA's last piece of the group: take its tickets.  (Taking them one tile later, when the fence
      // would be free, was measured slower: it delays the finalize of every group.)
      __threadfence();
      __syncthreads();
      if (threadIdx.x == 0 && atomicAdd(&p.ctr[group], pending) + pending == p.expected[group]) {
        __threadfence();  // acquire: the other CTAs' pieces are visible to whatever follows the next barrier
        s_done[++s_done[0]] = group;
      }
      pending = 0;
    }
  }
};

constexpr int kMaxDone = 62;

// FULL: Kd is a multiple of 1024, every segment's rows a multiple of 128, so the streaming loop carries
// no bounds predicates (padded token rows read row 0 and are never used).
template <int NT, bool HAS_LO, int PF, bool FULL>
__global__ void __launch_bounds__(512, (NT == 1 ? 2 : 1)) gemm_rows_kernel(const __grid_constant__ GemmArgs p) {
  constexpr int NW = 16, RB = (NT <= 4) ? 2 : 1;
  extern __shared__ __align__(16) float red[];  // [RB][NW][16][MP]
  __shared__ float sh[32];
  __shared__ float s_rstd[128];
  __shared__ int s_done[kMaxDone + 2];
  __shared__ int s_pos[128];
  __shared__ GroupMeta s_meta[kMetaSlots];
  const int c = blockIdx.x, G = gridDim.x;
  if (threadIdx.x == 0) s_done[0] = 0;
  if (p.epi.mode == EPI_QKV && threadIdx.x < p.s.M) {
    // inputs of the step and init-time constants: nothing an earlier kernel of this step writes
    s_pos[threadIdx.x] = p.epi.seq_lens[threadIdx.x / p.epi.K] + threadIdx.x % p.epi.K;
    s_rstd[threadIdx.x] = p.epi.rstd_mask[0];  // <mask> rows; fresh rows are overwritten in the finalize
  }
  const long long u0 = ((long long)c * p.U) / G, u1 = ((long long)(c + 1) * p.U) / G;
  int cand[kMetaSlots] = {-1, -1};  // groups whose piece tables sit in s_meta
  if (u0 < u1) {
    const int t0 = (int)(u0 / p.s.KR) >> 3, t1 = (int)((u1 - 1) / p.s.KR) >> 3;
    cand[0] = p.pair_offset > 0 ? t0 % p.pair_offset : t0;
    cand[1] = p.pair_offset > 0 ? t1 % p.pair_offset : t1;
    meta_prefetch(p, cand[0], &s_meta[0]);
    if (cand[1] != cand[0]) meta_prefetch(p, cand[1], &s_meta[1]);
  }
  __syncthreads();
  if (u0 < u1) {
    GemmEpi<NT, NW> epi{p, red, s_done, c, (int)(u0 / p.s.KR), 0};
    stream_units<NT, HAS_LO, PF, NW, RB, FULL>(p.s, u0, u1, red, epi);
  } else {
    pdl_wait();
  }
  pdl_trigger();
  __syncthreads();
  if (p.epi.mode == EPI_FC)
    for (int ftok = c; ftok < p.s.M; ftok += G) embed_rows(p, sh, ftok);
  // fused finalize of the groups this CTA completed (the streaming buffers are free now)
  const int n_done = s_done[0];
  FinSmem* fs = reinterpret_cast<FinSmem*>(red);
  asm volatile("cp.async.wait_all;" ::: "memory");
  __syncthreads();
  for (int i = 0; i < n_done; ++i) {
    const int group = s_done[1 + i];
    int slot = group == cand[0] ? 0 : (group == cand[1] ? 1 : -1);
    if (slot < 0) {  // a range that touches more than two groups (short reductions): fetch the table now
      slot = 0;
      cand[0] = group;
      meta_prefetch(p, group, &s_meta[0]);
      asm volatile("cp.async.wait_all;" ::: "memory");
      __syncthreads();
    }
    finalize_group<512, 0>(threadIdx.x, p, group, 8 * NT, sh, s_rstd, s_pos, &s_meta[slot], fs);
    if (threadIdx.x == 0) p.ctr[group] = 0;
    __syncthreads();
  }
}

// The <mask> rows are the same for every sequence and every step: their z row ([m_g * gain_g (not yet
// normalised) ; RMSNorm(m_e)]) and the 1/rms of m_g are computed once, at init.
__global__ void __launch_bounds__(256) mask_row_kernel(const bf16* mask_vec, const bf16* norm_g, const bf16* norm_e, int h,
                                                       float eps, bf16* z_hi, bf16* z_lo, float* rstd_mask, float* mask_res) {
  __shared__ float sh[32];
  float sg = 0.f, se = 0.f;
  for (int n = threadIdx.x; n < h; n += blockDim.x) {
    const float g = __bfloat162float(mask_vec[n]), e = __bfloat162float(mask_vec[h + n]);
    sg += g * g;
    se += e * e;
  }
  sg = block_sum(sg, sh);
  se = block_sum(se, sh);
  const float re = 1.f / sqrtf(se / (float)h + eps);
  if (threadIdx.x == 0) rstd_mask[0] = 1.f / sqrtf(sg / (float)h + eps);
  for (int n = threadIdx.x; n < h; n += blockDim.x) {
    bf16 hi, lo;
    split_bf16(__bfloat162float(mask_vec[n]) * __bfloat162float(norm_g[n]), hi, lo);
    z_hi[n] = hi; z_lo[n] = lo;
    mask_res[n] = __bfloat162float(mask_vec[n]);
    split_bf16(__bfloat162float(mask_vec[h + n]) * re * __bfloat162float(norm_e[n]), hi, lo);
    z_hi[h + n] = hi; z_lo[h + n] = lo;
  }
}

// (cos, sin) of every (position, frequency) pair the cache can hold, computed once in double precision.
__global__ void rope_table_kernel(float2* tab, int n_pos, int half, double theta, int dh) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)n_pos * half) return;
  const int pos = (int)(idx / half), i = (int)(idx % half);
  const double inv = pow(theta, -2.0 * (double)i / (double)dh);
  double sn, cs;
  sincos((double)pos * inv, &sn, &cs);
  tab[idx] = make_float2((float)cs, (float)sn);
}

cudaError_t launch_rope_table(float2* tab, int n_pos, int dh, float theta, cudaStream_t st) {
  const long long n = (long long)n_pos * (dh / 2);
  rope_table_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(tab, n_pos, dh / 2, (double)theta, dh);
  return cudaGetLastError();
}

__global__ void fill_mask_rows_kernel(bf16* z_hi, bf16* z_lo, const bf16* zmask_hi, const bf16* zmask_lo, int K, const FreshOffsets foff,
                                      int width) {
  const int tok = blockIdx.x, b = tok / K;
  if (tok % K < foff.v[b + 1] - foff.v[b]) return;
  const uint4* sh = reinterpret_cast<const uint4*>(zmask_hi);
  const uint4* sl = reinterpret_cast<const uint4*>(zmask_lo);
  uint4* dh = reinterpret_cast<uint4*>(z_hi + (size_t)tok * width);
  uint4* dl = reinterpret_cast<uint4*>(z_lo + (size_t)tok * width);
  for (int i = threadIdx.x; i < width / 8; i += blockDim.x) { dh[i] = sh[i]; dl[i] = sl[i]; }
}

cudaError_t launch_fill_mask_rows(bf16* z_hi, bf16* z_lo, const bf16* zmask_hi, const bf16* zmask_lo, int B, int K,
                                  const FreshOffsets& foff, int width, cudaStream_t st) {
  fill_mask_rows_kernel<<<B * K, 256, 0, st>>>(z_hi, z_lo, zmask_hi, zmask_lo, K, foff, width);
  return cudaGetLastError();
}

// Pre-fused features (feat_in = 0): the caller hands g [fresh rows][h] itself, so the feature FC is skipped and
// this kernel does what its prologue and epilogue do for one fresh row per block (Section 3.2): the residual
// g as fp32, z's g half = hi/lo of g * gain, the sums of squares of g per 128-column tile (the 1/rms is applied
// after the QKV projection), and z's e half = RMSNorm of the next token's embedding.
__global__ void __launch_bounds__(128) prefused_rows_kernel(const EpiArgs e, const bf16* __restrict__ g, int MP) {
  __shared__ float sh[32];
  const int t = blockIdx.x, tid = threadIdx.x;
  pdl_wait();
  const int orow = fresh_to_step_row(e, t);
  const bf16* grow = g + (size_t)t * e.h;
  for (int n0 = 0, tile = 0; n0 < e.h; n0 += 128, ++tile) {
    const int n = n0 + tid;
    float x = 0.f;
    if (n < e.h) {
      x = __bfloat162float(grow[n]);
      e.res0[(size_t)t * e.h + n] = x;
      bf16 hi, lo;
      split_bf16(x * __bfloat162float(e.gamma[n]), hi, lo);
      e.out_hi[(size_t)orow * e.ld_out + n] = hi;
      e.out_lo[(size_t)orow * e.ld_out + n] = lo;
    }
    const float ss = block_sum(x * x, sh);
    if (tid == 0) e.ss_out[(size_t)tile * MP + t] = ss;
  }
  // the shifted token embedding of this fresh row
  const int id = min(max(e.tokens[t], 0), e.vocab - 1);
  const bf16* row = e.embed + (size_t)id * e.h;
  float ss = 0.f;
  for (int n = tid; n < e.h; n += 128) {
    const float v = __bfloat162float(row[n]);
    ss += v * v;
  }
  ss = block_sum(ss, sh);
  const float rs = 1.f / sqrtf(ss / (float)e.h + e.eps);
  for (int n = tid; n < e.h; n += 128) {
    bf16 hi, lo;
    split_bf16(__bfloat162float(row[n]) * rs * __bfloat162float(e.gamma_e[n]), hi, lo);
    e.out_hi[(size_t)orow * e.ld_out + e.h + n] = hi;
    e.out_lo[(size_t)orow * e.ld_out + e.h + n] = lo;
  }
}

cudaError_t launch_prefused_rows(const EpiArgs& e, const bf16* g, int n_fresh, cudaStream_t st) {
  return launch_pdl(prefused_rows_kernel, dim3(n_fresh), dim3(128), 0, st, e, g, padded_tokens(n_fresh));
}

cudaError_t launch_mask_row(const bf16* mask_vec, const bf16* norm_g, const bf16* norm_e, int h, float eps, bf16* z_hi,
                            bf16* z_lo, float* rstd_mask, float* mask_res, cudaStream_t st) {
  mask_row_kernel<<<1, 256, 0, st>>>(mask_vec, norm_g, norm_e, h, eps, z_hi, z_lo, rstd_mask, mask_res);
  return cudaGetLastError();
}

template <int NT, bool HAS_LO, int PF>
static cudaError_t launch_t(const GemmArgs& a, int grid, bool full, cudaStream_t st) {
  constexpr int RB = (NT <= 4) ? 2 : 1;
  const size_t smem = (size_t)RB * 16 * 16 * 8 * NT * sizeof(float);
  cudaError_t e;
  if (full) {
    if (smem > 48 * 1024 && (e = cudaFuncSetAttribute(gemm_rows_kernel<NT, HAS_LO, PF, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    return launch_pdl(gemm_rows_kernel<NT, HAS_LO, PF, true>, dim3(grid), dim3(512), smem, st, a);
  } else {
    if (smem > 48 * 1024 && (e = cudaFuncSetAttribute(gemm_rows_kernel<NT, HAS_LO, PF, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    return launch_pdl(gemm_rows_kernel<NT, HAS_LO, PF, false>, dim3(grid), dim3(512), smem, st, a);
  }
}

cudaError_t launch_gemm_rows(const GemmPlan& plan, const GemmInput& in, const EpiArgs& epi, float* part, cudaStream_t st) {
  GemmArgs a;
  for (int i = 0; i < 6; ++i) a.s.seg[i] = plan.seg[i < plan.nseg ? i : 0];
  a.s.nseg = plan.nseg;
  a.s.Kd = plan.Kd; a.s.SK = plan.SK; a.s.KR = plan.KR; a.slots = plan.slots; a.U = plan.U;
  a.s.x_hi = in.x_hi; a.s.x_lo = in.x_lo != nullptr ? in.x_lo : in.x_hi; a.s.ldx = in.ldx; a.s.M = in.M;
  a.part = part; a.meta = plan.d_meta; a.meta_stride = plan.meta_stride;
  a.ctr = plan.d_ctr; a.expected = plan.d_expected; a.pair_offset = plan.pair_offset;
  a.epi = epi;
  const int MP = padded_tokens(in.M);
  const bool lo = in.x_lo != nullptr;
  bool full = (plan.Kd % 1024 == 0);   // padded token rows are harmless: they read row 0 and are never used
  for (int i = 0; i < plan.nseg; ++i) full = full && (plan.seg[i].rows % 128 == 0);
  #ifndef DART_GEMM_PF
#define DART_GEMM_PF 1
#endif
  if (MP == 8) return lo ? launch_t<1, true, DART_GEMM_PF>(a, plan.grid, full, st) : launch_t<1, false, DART_GEMM_PF>(a, plan.grid, full, st);
  if (MP == 32) return lo ? launch_t<4, true, 2>(a, plan.grid, full, st) : launch_t<4, false, 2>(a, plan.grid, full, st);
  return lo ? launch_t<16, true, 1>(a, plan.grid, full, st) : launch_t<16, false, 1>(a, plan.grid, full, st);
}

}  // namespace dart
