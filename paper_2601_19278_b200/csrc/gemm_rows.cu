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

namespace dart {

// ------------------------------------------------------------------------------------------
// Fused epilogues, run by the CTA that completes a tile (or a pair of tiles).
// ------------------------------------------------------------------------------------------
// Shared-memory description of one group: for each of its (up to 16) 16-row tiles, the partial pieces
// to add up, as offsets into `part` in units of one 16 x MP piece, in CTA order.
constexpr int kMaxPieces = 33;
struct GroupMeta {
  int cnt[16];
  unsigned off[16][kMaxPieces];
};

__device__ __forceinline__ void load_group_meta(const GemmArgs& p, int Ta, int Tb, bool paired, GroupMeta* gm) {
  const int j = threadIdx.x;
  if (j < 16 && (j < 8 || paired)) {
    const int mt = (j < 8 ? Ta : Tb) * 8 + (j & 7);
    const int lo = p.clo[mt], hi = p.chi[mt];
    int n = 0;
    for (int c = lo; c <= hi && n < kMaxPieces; ++c) gm->off[j][n++] = (unsigned)(c * p.slots + (mt - p.first_mt[c]));
    gm->cnt[j] = n;
  }
  __syncthreads();
}

// which: 0 = tile Ta, 1 = tile Tb of the group
__device__ __forceinline__ float piece_sum(const GemmArgs& p, const GroupMeta* gm, int which, int row, int tok, int MP) {
  float s = 0.f;
  const int j = which * 8 + (row >> 4), r = row & 15;
  const int n = gm->cnt[j];
  for (int i = 0; i < n; ++i) s += p.part[((size_t)gm->off[j][i] * 16 + r) * MP + tok];
  return s;
}

// 1/rms of every token row from per-tile sums of squares ss[tile][mp] (tiles of a width-`h` row), into
// s_rstd[0..M).  Four threads per token add up interleaved tiles, then their four partials are added in a
// fixed order.  col(tok) maps a token to its column of ss.  Needs M <= 128 and blockDim >= 512.
template <class ColFn>
__device__ __forceinline__ void rstd_all(const float* ss, int ntile, int mp, int M, int h, float eps, float* s_part,
                                         float* s_rstd, ColFn col) {
  const int tid = threadIdx.x;
  if (tid < 4 * M) {
    const int tok = tid >> 2, q = tid & 3;
    const int cidx = col(tok);
    float s = 0.f;
    if (cidx >= 0)
      for (int t = q; t < ntile; t += 4) s += ss[(size_t)t * mp + cidx];
    s_part[tid] = s;
  }
  __syncthreads();
  if (tid < M) {
    const float s = s_part[4 * tid] + s_part[4 * tid + 1] + s_part[4 * tid + 2] + s_part[4 * tid + 3];
    if (col(tid) >= 0) s_rstd[tid] = 1.f / sqrtf(s / (float)h + eps);
  }
  __syncthreads();
}

// sum over the group's 128 rows of v (one value per thread: row = tid & 127, token class = tid >> 7),
// result valid in every thread; fixed order.  sh: one float per warp.
__device__ __forceinline__ float tile_rows_sum(float v, float* sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) sh[warp] = v;
  __syncthreads();
  const int cls = warp >> 2;  // warps 4*cls .. 4*cls+3 hold the 128 rows of token class cls
  return sh[cls * 4] + sh[cls * 4 + 1] + sh[cls * 4 + 2] + sh[cls * 4 + 3];
}

__device__ __noinline__ void finalize_group(const GemmArgs& p, int group, int MP, float* sh, float* s_rstd, GroupMeta* gm,
                                            float* s_part) {
  const EpiArgs& e = p.epi;
  const int tid = threadIdx.x;
  const int Ta = group, Tb = group + p.pair_offset;
  load_group_meta(p, Ta, Tb, p.pair_offset > 0, gm);
  int s = 0;  // segment of tile Ta
  for (int i = 1; i < 6; ++i)
    if (i < p.s.nseg && Ta >= p.s.seg[i].tile0) s = i;
  const int row_base = (Ta - p.s.seg[s].tile0) * 128;       // first row of the tile inside its matrix
  const int rows_valid = min(128, p.s.seg[s].rows - row_base);
  const int row = tid & 127, par = tid >> 7;               // thread -> (row, token class)
  const int npar = blockDim.x >> 7;

  if (e.mode == EPI_FC) {
    // g = FC(features) on the fresh rows: residual stream, gain-scaled hi/lo, tile sum of squares
    for (int tok = par; tok < MP; tok += npar) {
      float g = 0.f;
      if (row < rows_valid && tok < p.s.M) g = piece_sum(p, gm, 0, row, tok, MP);
      const float ssq = tile_rows_sum(g * g, sh);
      if (row < rows_valid && tok < p.s.M) {
        const int n = row_base + row;
        e.res0[(size_t)tok * e.h + n] = g;
        bf16 hi, lo;
        split_bf16(g * __bfloat162float(e.gamma[n]), hi, lo);
        e.out_hi[(size_t)tok * e.ld_out + n] = hi;
        e.out_lo[(size_t)tok * e.ld_out + n] = lo;
      }
      if (row == 0 && tok < p.s.M) e.ss_out[(size_t)Ta * MP + tok] = ssq;
    }
  } else if (e.mode == EPI_RES) {
    // x = residual + proj; gain-scaled hi/lo for the next projection; tile sum of squares
    for (int tok = par; tok < MP; tok += npar) {
      float x = 0.f;
      if (row < rows_valid && tok < p.s.M) {
        const int n = row_base + row;
        float r;
        if (e.res_in != nullptr) r = e.res_in[(size_t)tok * e.h + n];
        else {  // first residual: g of a fresh row, or the <mask> representation
          const int b = tok / e.K, rr = tok % e.K;
          r = rr < e.F ? e.res0[(size_t)(b * e.F + rr) * e.h + n] : __bfloat162float(e.mask_vec[n]);
        }
        x = r + piece_sum(p, gm, 0, row, tok, MP);
      }
      const float ssq = tile_rows_sum(x * x, sh);
      if (row < rows_valid && tok < p.s.M) {
        const int n = row_base + row;
        if (e.res_out != nullptr) e.res_out[(size_t)tok * e.h + n] = x;
        bf16 hi, lo;
        split_bf16(x * __bfloat162float(e.gamma[n]), hi, lo);
        e.out_hi[(size_t)tok * e.ld_out + n] = hi;
        e.out_lo[(size_t)tok * e.ld_out + n] = lo;
      }
      if (row == 0 && tok < p.s.M) e.ss_out[(size_t)Ta * MP + tok] = ssq;
    }
  } else if (e.mode == EPI_GATE_UP) {
    // u = SiLU(rstd * gate) * (rstd * up): the previous RMSNorm's 1/rms is applied here
    rstd_all(e.ss_in, e.ss_tiles, e.ss_mp, p.s.M, e.h, e.eps, s_part, s_rstd, [](int tok) { return tok; });
    for (int tok = par; tok < p.s.M; tok += npar) {
      if (row < rows_valid) {
        const int n = row_base + row;
        const float gt = s_rstd[tok] * piece_sum(p, gm, 0, row, tok, MP);
        const float up = s_rstd[tok] * piece_sum(p, gm, 1, row, tok, MP);
        bf16 hi, lo;
        split_bf16(gt / (1.f + expf(-gt)) * up, hi, lo);
        e.out_hi[(size_t)tok * e.ld_out + n] = hi;
        e.out_lo[(size_t)tok * e.ld_out + n] = lo;
      }
    }
  } else if (e.mode == EPI_QKV) {
    // y = rstd_g * (W[:, :h] z_g) + W[:, h:] z_e ; RoPE on q, k at position P_b + r ; q and the new rows'
    // k, v as hi/lo pairs ; the fresh rows' k, v appended to the cache
    if (tid < p.s.M) s_rstd[tid] = e.rstd_mask[0];  // <mask> rows; fresh rows are overwritten below
    __syncthreads();
    {
      const int K = e.K, F = e.F;
      rstd_all(e.ss_in, e.ss_tiles, e.ss_mp, p.s.M, e.h, e.eps, s_part, s_rstd,
               [K, F](int tok) { const int b = tok / K, rr = tok % K; return rr < F ? b * F + rr : -1; });
    }
    const int kind = s;  // segment 0,1,2 = q,k,v (g half); the e half is the paired tile
    const int dh = e.dh, half = dh >> 1;
    const int pairs = (rows_valid / dh) * half;  // (head, i) pairs in this tile
    for (int idx = tid; idx < pairs * p.s.M; idx += blockDim.x) {
      const int tok = idx / pairs, pi = idx - tok * pairs;
      const int hl = pi / half, i = pi - hl * half;
      const int ra = hl * dh + i, rb = ra + half;
      const float x1 = s_rstd[tok] * piece_sum(p, gm, 0, ra, tok, MP) + piece_sum(p, gm, 1, ra, tok, MP);
      const float x2 = s_rstd[tok] * piece_sum(p, gm, 0, rb, tok, MP) + piece_sum(p, gm, 1, rb, tok, MP);
      const int b = tok / e.K, r = tok % e.K;
      const long long pos = (long long)e.seq_lens[b] + r;
      float o1 = x1, o2 = x2;
      if (kind < 2) {
        const double inv = pow((double)e.rope_theta, -2.0 * (double)i / (double)dh);
        double sn, cs;
        sincos((double)pos * inv, &sn, &cs);
        o1 = (float)((double)x1 * cs - (double)x2 * sn);
        o2 = (float)((double)x2 * cs + (double)x1 * sn);
      }
      bf16 h1, l1, h2, l2;
      split_bf16(o1, h1, l1);
      split_bf16(o2, h2, l2);
      const int head = (row_base / dh) + hl;
      if (kind == 0) {
        const size_t o = (((size_t)b * e.Hq + head) * e.K + r) * dh;
        e.q_hi[o + i] = h1; e.q_hi[o + i + half] = h2;
        e.q_lo[o + i] = l1; e.q_lo[o + i + half] = l2;
      } else {
        bf16* side = (kind == 1 ? e.k_new : e.v_new) + ((size_t)b * e.Hkv + head) * 16 * dh;
        side[(size_t)r * dh + i] = h1; side[(size_t)r * dh + i + half] = h2;
        side[(size_t)(8 + r) * dh + i] = l1; side[(size_t)(8 + r) * dh + i + half] = l2;
        if (r < e.F) {
          bf16* dst = (kind == 1 ? e.k_cache : e.v_cache) + (((size_t)b * e.Hkv + head) * e.P_cap + pos) * dh;
          dst[i] = h1;
          dst[i + half] = h2;
        }
      }
    }
  }
}

// Shifted token embedding of the fresh rows (Section 3.2): e = E[token], normalised (its 1/rms needs
// nothing else) and written as the second half of the fresh row's z.  One CTA per fresh row.
__device__ __noinline__ void embed_rows(const GemmArgs& p, float* sh) {
  const EpiArgs& e = p.epi;
  const int ftok = blockIdx.x;
  const int id = min(max(e.tokens[ftok], 0), e.vocab - 1);
  const bf16* row = e.embed + (size_t)id * e.h;
  float ss = 0.f;
  for (int n = threadIdx.x; n < e.h; n += blockDim.x) {
    const float v = __bfloat162float(row[n]);
    ss += v * v;
  }
  ss = block_sum(ss, sh);
  const float rs = 1.f / sqrtf(ss / (float)e.h + e.eps);
  for (int n = threadIdx.x; n < e.h; n += blockDim.x) {
    bf16 hi, lo;
    split_bf16(__bfloat162float(row[n]) * rs * __bfloat162float(e.gamma_e[n]), hi, lo);
    e.out_hi[(size_t)ftok * e.ld_out + e.h + n] = hi;
    e.out_lo[(size_t)ftok * e.ld_out + e.h + n] = lo;
  }
}

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
      // this CTA's last piece of the group: take its tickets
      __threadfence();
      __syncthreads();
      if (threadIdx.x == 0 && atomicAdd(&p.ctr[group], pending) + pending == p.expected[group]) s_done[++s_done[0]] = group;
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
  const int c = blockIdx.x, G = gridDim.x;
  if (threadIdx.x == 0) s_done[0] = 0;
  const long long u0 = ((long long)c * p.U) / G, u1 = ((long long)(c + 1) * p.U) / G;
  __syncthreads();
  if (u0 < u1) {
    GemmEpi<NT, NW> epi{p, red, s_done, c, (int)(u0 / p.s.KR), 0};
    stream_units<NT, HAS_LO, PF, NW, RB, FULL>(p.s, u0, u1, red, epi);
  } else {
    pdl_wait();
  }
  pdl_trigger();
  __syncthreads();
  if (p.epi.mode == EPI_FC && c < p.s.M) embed_rows(p, sh);
  // fused finalize of the groups this CTA completed (the streaming buffers are free now)
  const int n_done = s_done[0];
  GroupMeta* gm = reinterpret_cast<GroupMeta*>(red);
  float* s_part = reinterpret_cast<float*>(gm + 1);
  for (int i = 0; i < n_done; ++i) {
    const int group = s_done[1 + i];
    __threadfence();
    finalize_group(p, group, 8 * NT, sh, s_rstd, gm, s_part);
    if (threadIdx.x == 0) p.ctr[group] = 0;
    __syncthreads();
  }
}

// The <mask> rows are the same for every sequence and every step: their z row ([m_g * gain_g (not yet
// normalised) ; RMSNorm(m_e)]) and the 1/rms of m_g are computed once, at init.
__global__ void __launch_bounds__(256) mask_row_kernel(const bf16* mask_vec, const bf16* norm_g, const bf16* norm_e, int h,
                                                       float eps, bf16* z_hi, bf16* z_lo, float* rstd_mask) {
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
    split_bf16(__bfloat162float(mask_vec[h + n]) * re * __bfloat162float(norm_e[n]), hi, lo);
    z_hi[h + n] = hi; z_lo[h + n] = lo;
  }
}

cudaError_t launch_mask_row(const bf16* mask_vec, const bf16* norm_g, const bf16* norm_e, int h, float eps, bf16* z_hi,
                            bf16* z_lo, float* rstd_mask, cudaStream_t st) {
  mask_row_kernel<<<1, 256, 0, st>>>(mask_vec, norm_g, norm_e, h, eps, z_hi, z_lo, rstd_mask);
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
  a.s.x_K = in.x_K; a.s.x_F = in.x_F; a.s.x_mask_row = in.x_mask_row;
  a.part = part; a.first_mt = plan.d_first_mt; a.clo = plan.d_mt_clo; a.chi = plan.d_mt_chi;
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
