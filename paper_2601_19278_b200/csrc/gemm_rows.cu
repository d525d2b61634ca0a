// Weight-streaming small-M GEMM for the draft layer's projections (FC, QKV, o_proj, gate/up,
// down -- Section 3.2's single decoder layer) with the op that follows each projection fused
// into its epilogue.
//
// The op is HBM-bound: M = batch*K token rows (8..128) against weight matrices of 10^7..10^8
// elements, i.e. M flop per weight byte.  Design:
//   * weights are the MMA's M-side operand (16 weight rows x 16 k per mma.sync.m16n8k16),
//     token rows are the 8-wide N side, so M = 8 tokens is an exact fit;
//   * weight fragments go global -> registers with 128-bit loads; the k index is permuted
//     identically on both operands so that the 2 x 16 bytes a thread loads are exactly its
//     fragment slots;
//   * activations (a few hundred KB, bf16 hi + lo) are read through L1 by every warp;
//   * the flattened (128-row tile, 64-wide k-step) space is cut into gridDim.x equal ranges,
//     so every CTA streams the same number of bytes (no tail wave).  A CTA writes one fp32
//     partial per tile it touches and takes a ticket on the tile's counter; the CTA that takes
//     the last ticket sums the tile's partials in CTA order (deterministic, no float atomics)
//     and applies the fused op: residual add, RMSNorm gain + sum of squares, RoPE + cache
//     append, or SiLU-gate.
//   * RMSNorm's 1/rms is a per-token scalar, so it is applied *after* the next projection
//     (W (x*gain) * rstd): no row-wide reduction ever sits between two kernels.  A finalizer
//     only emits its tile's partial sum of squares; whoever needs rstd adds up the tiles'.
#include "common.cuh"
#include "kernels.h"

namespace dart {

struct RowCursor {
  int tile, ks;
  const bf16* r0;
  const bf16* r1;
  int xoff;
  bool valid;
  __device__ __forceinline__ void set_tile(const GemmArgs& p, int warp, int g) {
    int s = 0;
#pragma unroll
    for (int i = 1; i < 6; ++i)
      if (i < p.nseg && tile >= p.seg[i].tile0) s = i;
    const GemmSeg sg = p.seg[s];
    const int row0 = (tile - sg.tile0) * 128 + warp * 16;
    valid = row0 < sg.rows;
    r0 = sg.W + (size_t)(valid ? row0 + g : 0) * sg.ld;
    r1 = r0 + (size_t)(valid ? 8 : 0) * sg.ld;
    xoff = sg.xoff;
  }
  __device__ __forceinline__ void advance(const GemmArgs& p, int warp, int g) {
    if (++ks == p.SK) {
      ks = 0;
      ++tile;
      set_tile(p, warp, g);
    }
  }
};

// ------------------------------------------------------------------------------------------
// Fused epilogues, run by the CTA that completes a tile (or a pair of tiles).
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ float piece_sum(const GemmArgs& p, int tile, int row, int tok, int MP) {
  float s = 0.f;
  const int lo = p.clo[tile], hi = p.chi[tile];
  for (int c = lo; c <= hi; ++c)
    s += p.part[(((size_t)c * p.slots + (tile - p.first_tile[c])) * 128 + row) * MP + tok];
  return s;
}

// rstd of a token from per-tile sums of squares ss[tile][mp] over `ntile` tiles of a width-`h` row
__device__ __forceinline__ float rstd_from(const float* ss, int ntile, int mp, int col, int h, float eps) {
  float s = 0.f;
  for (int t = 0; t < ntile; ++t) s += ss[(size_t)t * mp + col];
  return 1.f / sqrtf(s / (float)h + eps);
}

// sum over the tile's 128 rows of v (one value per thread: row = tid & 127, token parity = tid >> 7),
// result valid in every thread; fixed order.  sh: 8 floats.
__device__ __forceinline__ float tile_rows_sum(float v, float* sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) sh[warp] = v;
  __syncthreads();
  const int half = warp >> 2;  // warps 0..3 hold token parity 0, warps 4..7 parity 1
  return sh[half * 4] + sh[half * 4 + 1] + sh[half * 4 + 2] + sh[half * 4 + 3];
}

__device__ void finalize_group(const GemmArgs& p, int group, int MP, float* sh, float* s_rstd) {
  const EpiArgs& e = p.epi;
  const int tid = threadIdx.x;
  const int Ta = group, Tb = group + p.pair_offset;
  int s = 0;  // segment of tile Ta
  for (int i = 1; i < 6; ++i)
    if (i < p.nseg && Ta >= p.seg[i].tile0) s = i;
  const int row_base = (Ta - p.seg[s].tile0) * 128;       // first row of the tile inside its matrix
  const int rows_valid = min(128, p.seg[s].rows - row_base);
  const int row = tid & 127, par = tid >> 7;               // thread -> (row, token parity)

  if (e.mode == EPI_FC) {
    // g = FC(features) on the fresh rows: residual stream, gain-scaled hi/lo, tile sum of squares
    for (int tok = par; tok < MP; tok += 2) {
      float g = 0.f;
      if (row < rows_valid && tok < p.M) g = piece_sum(p, Ta, row, tok, MP);
      const float ssq = tile_rows_sum(g * g, sh);
      if (row < rows_valid && tok < p.M) {
        const int n = row_base + row;
        e.res0[(size_t)tok * e.h + n] = g;
        bf16 hi, lo;
        split_bf16(g * __bfloat162float(e.gamma[n]), hi, lo);
        e.out_hi[(size_t)tok * e.ld_out + n] = hi;
        e.out_lo[(size_t)tok * e.ld_out + n] = lo;
      }
      if (row == 0 && tok < p.M) e.ss_out[(size_t)Ta * MP + tok] = ssq;
    }
  } else if (e.mode == EPI_RES) {
    // x = residual + proj; gain-scaled hi/lo for the next projection; tile sum of squares
    for (int tok = par; tok < MP; tok += 2) {
      float x = 0.f;
      if (row < rows_valid && tok < p.M) {
        const int n = row_base + row;
        float r;
        if (e.res_in != nullptr) r = e.res_in[(size_t)tok * e.h + n];
        else {  // first residual: g of a fresh row, or the <mask> representation
          const int b = tok / e.K, rr = tok % e.K;
          r = rr < e.F ? e.res0[(size_t)(b * e.F + rr) * e.h + n] : __bfloat162float(e.mask_vec[n]);
        }
        x = r + piece_sum(p, Ta, row, tok, MP);
      }
      const float ssq = tile_rows_sum(x * x, sh);
      if (row < rows_valid && tok < p.M) {
        const int n = row_base + row;
        if (e.res_out != nullptr) e.res_out[(size_t)tok * e.h + n] = x;
        bf16 hi, lo;
        split_bf16(x * __bfloat162float(e.gamma[n]), hi, lo);
        e.out_hi[(size_t)tok * e.ld_out + n] = hi;
        e.out_lo[(size_t)tok * e.ld_out + n] = lo;
      }
      if (row == 0 && tok < p.M) e.ss_out[(size_t)Ta * MP + tok] = ssq;
    }
  } else if (e.mode == EPI_GATE_UP) {
    // u = SiLU(rstd * gate) * (rstd * up): the previous RMSNorm's 1/rms is applied here
    if (tid < p.M) s_rstd[tid] = rstd_from(e.ss_in, e.ss_tiles, e.ss_mp, tid, e.h, e.eps);
    __syncthreads();
    for (int tok = par; tok < p.M; tok += 2) {
      if (row < rows_valid) {
        const int n = row_base + row;
        const float gt = s_rstd[tok] * piece_sum(p, Ta, row, tok, MP);
        const float up = s_rstd[tok] * piece_sum(p, Tb, row, tok, MP);
        bf16 hi, lo;
        split_bf16(gt / (1.f + expf(-gt)) * up, hi, lo);
        e.out_hi[(size_t)tok * e.ld_out + n] = hi;
        e.out_lo[(size_t)tok * e.ld_out + n] = lo;
      }
    }
  } else if (e.mode == EPI_QKV) {
    // y = rstd_g * (W[:, :h] z_g) + W[:, h:] z_e ; RoPE on q, k at position P_b + r ; q and the new rows'
    // k, v as hi/lo pairs ; the fresh rows' k, v appended to the cache
    if (tid < p.M) {
      const int b = tid / e.K, rr = tid % e.K;
      s_rstd[tid] = rr < e.F ? rstd_from(e.ss_in, e.ss_tiles, e.ss_mp, b * e.F + rr, e.h, e.eps) : e.rstd_mask[0];
    }
    __syncthreads();
    const int kind = s;  // segment 0,1,2 = q,k,v (g half); the e half is the paired tile
    const int dh = e.dh, half = dh >> 1;
    const int pairs = (rows_valid / dh) * half;  // (head, i) pairs in this tile
    for (int idx = tid; idx < pairs * p.M; idx += 256) {
      const int tok = idx / pairs, pi = idx - tok * pairs;
      const int hl = pi / half, i = pi - hl * half;
      const int ra = hl * dh + i, rb = ra + half;
      const float x1 = s_rstd[tok] * piece_sum(p, Ta, ra, tok, MP) + piece_sum(p, Tb, ra, tok, MP);
      const float x2 = s_rstd[tok] * piece_sum(p, Ta, rb, tok, MP) + piece_sum(p, Tb, rb, tok, MP);
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
__device__ void embed_rows(const GemmArgs& p, float* sh) {
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

// FULL: Kd is a multiple of 64, every segment's rows a multiple of 128 and all MP token rows are
// valid, so the streaming loop carries no bounds predicates.
template <int NT, bool HAS_LO, int PF, bool FULL>
__global__ void __launch_bounds__(256, (NT <= 4 ? 2 : 1)) gemm_rows_kernel(const GemmArgs p) {
  constexpr int MP = 8 * NT;
  __shared__ float sh[32];
  __shared__ float s_rstd[128];
  __shared__ int s_last;
  const int c = blockIdx.x, G = gridDim.x;
  if (p.epi.mode == EPI_FC && c < p.M) embed_rows(p, sh);
  const long long u0 = ((long long)c * p.U) / G, u1 = ((long long)(c + 1) * p.U) / G;
  if (u0 >= u1) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int tile_first = (int)(u0 / p.SK);

  float acc[NT][4];
#pragma unroll
  for (int n = 0; n < NT; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
  uint4 a[PF][4];

  // activation row of each token this thread feeds to the MMA (token n*8+g); with x_K > 0 the rows
  // r >= x_F of every sequence all read the shared <mask> row
  const bf16* xh[NT];
  const long long xlo_delta = p.x_lo - p.x_hi;
#pragma unroll
  for (int n = 0; n < NT; ++n) {
    const int tok = n * 8 + g;
    long long rowi = tok;
    if (p.x_K > 0) {
      const int b = tok / p.x_K, r = tok % p.x_K;
      rowi = r < p.x_F ? (long long)b * p.x_F + r : p.x_mask_row;
    }
    xh[n] = p.x_hi + rowi * p.ldx;
  }

  RowCursor ld, cp;
  ld.tile = cp.tile = tile_first;
  ld.ks = cp.ks = (int)(u0 - (long long)tile_first * p.SK);
  ld.set_tile(p, warp, g);
  cp.set_tile(p, warp, g);

  auto issue = [&](uint4(&dst)[4]) {
    const int ka = ld.ks * 64 + chunk_k0(t), kb = ld.ks * 64 + chunk_k1(t);
    if (FULL) {
      dst[0] = ld_stream16(ld.r0 + ka);
      dst[1] = ld_stream16(ld.r0 + kb);
      dst[2] = ld_stream16(ld.r1 + ka);
      dst[3] = ld_stream16(ld.r1 + kb);
    } else {
      const bool va = ld.valid && ka < p.Kd, vb = ld.valid && kb < p.Kd;
      const uint4 z = make_uint4(0, 0, 0, 0);
      dst[0] = va ? ld_stream16(ld.r0 + ka) : z;
      dst[1] = vb ? ld_stream16(ld.r0 + kb) : z;
      dst[2] = va ? ld_stream16(ld.r1 + ka) : z;
      dst[3] = vb ? ld_stream16(ld.r1 + kb) : z;
    }
    ld.advance(p, warp, g);
  };

#pragma unroll
  for (int s = 0; s < PF; ++s)
    if (u0 + s < u1) issue(a[s]);

  for (long long u = u0; u < u1; u += PF) {
#pragma unroll
    for (int s = 0; s < PF; ++s) {
      if (u + s < u1) {
        const int ka = cp.ks * 64 + chunk_k0(t), kb = cp.ks * 64 + chunk_k1(t);
        const bool kval = ka < p.Kd, kval2 = kb < p.Kd;
        const uint32_t w0[8] = {a[s][0].x, a[s][0].y, a[s][0].z, a[s][0].w, a[s][1].x, a[s][1].y, a[s][1].z, a[s][1].w};
        const uint32_t w1[8] = {a[s][2].x, a[s][2].y, a[s][2].z, a[s][2].w, a[s][3].x, a[s][3].y, a[s][3].z, a[s][3].w};
#pragma unroll
        for (int n = 0; n < NT; ++n) {
          const int tok = n * 8 + g;
          uint4 h0 = make_uint4(0, 0, 0, 0), h1 = h0, l0 = h0, l1 = h0;
          const bf16* xp = xh[n] + cp.xoff;
          const bf16* xq = xp + xlo_delta;
          if (FULL) {
            h0 = ld_act16(xp + ka);
            h1 = ld_act16(xp + kb);
            if (HAS_LO) { l0 = ld_act16(xq + ka); l1 = ld_act16(xq + kb); }
          } else if (tok < p.M) {
            if (kval) {
              h0 = ld_act16(xp + ka);
              if (HAS_LO) l0 = ld_act16(xq + ka);
            }
            if (kval2) {
              h1 = ld_act16(xp + kb);
              if (HAS_LO) l1 = ld_act16(xq + kb);
            }
          }
          const uint32_t xhv[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
          const uint32_t xlv[8] = {l0.x, l0.y, l0.z, l0.w, l1.x, l1.y, l1.z, l1.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            mma_bf16_16816(acc[n], w0[2 * j], w1[2 * j], w0[2 * j + 1], w1[2 * j + 1], xhv[2 * j], xhv[2 * j + 1]);
            if (HAS_LO)
              mma_bf16_16816(acc[n], w0[2 * j], w1[2 * j], w0[2 * j + 1], w1[2 * j + 1], xlv[2 * j], xlv[2 * j + 1]);
          }
        }
        if (u + s + PF < u1) issue(a[s]);
        const bool tile_end = (cp.ks == p.SK - 1) || (u + s == u1 - 1);
        if (tile_end) {
          if (cp.valid) {
            float* dst = p.part + (((size_t)c * p.slots + (cp.tile - tile_first)) * 128 + warp * 16) * MP;
#pragma unroll
            for (int n = 0; n < NT; ++n) {
              *reinterpret_cast<float2*>(dst + (size_t)g * MP + n * 8 + 2 * t) = make_float2(acc[n][0], acc[n][1]);
              *reinterpret_cast<float2*>(dst + (size_t)(g + 8) * MP + n * 8 + 2 * t) = make_float2(acc[n][2], acc[n][3]);
            }
          }
#pragma unroll
          for (int n = 0; n < NT; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
          // ticket: the CTA that completes the tile (pair) runs the fused epilogue
          const int group = p.pair_offset > 0 ? cp.tile % p.pair_offset : cp.tile;
          __threadfence();
          __syncthreads();
          if (threadIdx.x == 0) s_last = (atomicAdd(&p.ctr[group], 1) == p.expected[group] - 1);
          __syncthreads();
          if (s_last) {
            __threadfence();
            finalize_group(p, group, MP, sh, s_rstd);
            if (threadIdx.x == 0) p.ctr[group] = 0;
          }
        }
        cp.advance(p, warp, g);
      }
    }
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
  if (full)
    gemm_rows_kernel<NT, HAS_LO, PF, true><<<grid, 256, 0, st>>>(a);
  else
    gemm_rows_kernel<NT, HAS_LO, PF, false><<<grid, 256, 0, st>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_gemm_rows(const GemmPlan& plan, const GemmInput& in, const EpiArgs& epi, float* part, cudaStream_t st) {
  GemmArgs a;
  for (int i = 0; i < 6; ++i) a.seg[i] = plan.seg[i < plan.nseg ? i : 0];
  a.nseg = plan.nseg;
  a.Kd = plan.Kd; a.SK = plan.SK; a.slots = plan.slots; a.U = plan.U;
  a.x_hi = in.x_hi; a.x_lo = in.x_lo != nullptr ? in.x_lo : in.x_hi; a.ldx = in.ldx; a.M = in.M;
  a.x_K = in.x_K; a.x_F = in.x_F; a.x_mask_row = in.x_mask_row;
  a.part = part; a.first_tile = plan.d_first_tile; a.clo = plan.d_tile_clo; a.chi = plan.d_tile_chi;
  a.ctr = plan.d_ctr; a.expected = plan.d_expected; a.pair_offset = plan.pair_offset;
  a.epi = epi;
  const int MP = padded_tokens(in.M);
  const bool lo = in.x_lo != nullptr;
  bool full = (plan.Kd % 64 == 0) && (in.M == MP);
  for (int i = 0; i < plan.nseg; ++i) full = full && (plan.seg[i].rows % 128 == 0);
  if (MP == 8) return lo ? launch_t<1, true, 4>(a, plan.grid, full, st) : launch_t<1, false, 4>(a, plan.grid, full, st);
  if (MP == 32) return lo ? launch_t<4, true, 2>(a, plan.grid, full, st) : launch_t<4, false, 2>(a, plan.grid, full, st);
  return lo ? launch_t<16, true, 2>(a, plan.grid, full, st) : launch_t<16, false, 2>(a, plan.grid, full, st);
}

}  // namespace dart
