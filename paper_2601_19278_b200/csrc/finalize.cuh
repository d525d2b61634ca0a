// Fused epilogues of the projections (umma_gemm.cu): the CTA
// that completes a 128-row group (or a pair of groups) adds up the stream-K pieces and applies the step's
// elementwise work (Section 3.2: RMSNorm scales, RoPE, residual adds, SiLU gating, cache append).
#pragma once
#include "common.cuh"
#include "kernels.h"

namespace dart {

// Packed index of fresh row (b, r), or -1 for a <mask> row.
__device__ __forceinline__ int fresh_index(const EpiArgs& e, int b, int r) {
  return r < e.foff[b + 1] - e.foff[b] ? e.foff[b] + r : -1;
}
// Step row b*K + r of packed fresh row f (a scan over at most 32 sequences).
__device__ __forceinline__ int fresh_to_step_row(const EpiArgs& e, int f) {
  int b = 0;
  while (b + 1 < e.B && f >= e.foff[b + 1]) ++b;
  return b * e.K + (f - e.foff[b]);
}

// ------------------------------------------------------------------------------------------
// Fused epilogues, run by the CTA that completes a tile (or a pair of tiles).
// ------------------------------------------------------------------------------------------
// Shared-memory working set of one finalize.
struct FinSmem {
  float rpart[512];      // partial sums of squares for the 1/rms
  float xs[2][128][9];   // summed pieces: [tile of the pair][row][token of the chunk], padded against conflicts
};
static_assert(sizeof(FinSmem) <= 2 * 16 * 16 * 8 * sizeof(float), "the finalize working set must fit the streaming buffers");

// Piece table of one group in shared memory: for each of its (up to 16) 16-row tiles the count and the
// offsets (units of one 16 x MP piece, CTA order) of the pieces to add up.  The table is plan data, so a
// CTA copies the rows of the groups it may end up finalizing (those its range touches) with cp.async
// right at its start; by the time a finalize runs they have long arrived.
struct GroupMeta { int row[16][kMetaStride]; };
constexpr int kMetaSlots = 2;

__device__ __forceinline__ void meta_prefetch(const GemmArgs& p, int group, GroupMeta* gm) {
  const int Ta = group, Tb = group + p.pair_offset;
  const int nrow = p.pair_offset > 0 ? 16 : 8;
  for (int i = threadIdx.x; i < nrow * kMetaStride; i += blockDim.x) {
    const int j = i / kMetaStride, q = i - j * kMetaStride;
    const int* src = p.meta + (size_t)((j < 8 ? Ta : Tb) * 8 + (j & 7)) * kMetaStride + q;
    const unsigned dst = (unsigned)__cvta_generic_to_shared(&gm->row[j][q]);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
}

// The finalize runs on a team of NTHR threads that synchronises on barrier BAR (0 = __syncthreads, NTHR = the
// whole CTA; a 256-thread team of otherwise idle warps was measured slower).
// ft is the thread's index in the team.
template <int NTHR, int BAR>
__device__ __forceinline__ void team_sync() {
  if (BAR == 0) __syncthreads();
  else asm volatile("bar.sync %0, %1;" ::"n"(BAR), "n"(NTHR) : "memory");
}

// Partial sum of squares of token row ft / TPT over the tiles q, q + TPT, ... (TPT = NTHR / MP threads
// per token); col(tok) maps a token to its column of ss[tile][mp], or -1.
template <int NTHR, class ColFn>
__device__ __forceinline__ float rstd_issue(int ft, const float* ss, int ntile, int mp, int M, int MP, ColFn col) {
  const int TPT = NTHR / MP, tok = ft / TPT, q = ft % TPT;
  const int cidx = tok < M ? col(tok) : -1;
  float s = 0.f;
  if (cidx >= 0) {
#pragma unroll 4
    for (int t = q; t < ntile; t += TPT) s += __ldcg(ss + (size_t)t * mp + cidx);
  }
  return s;
}
// Fixed-order reduction of those partials to s_rstd[tok] = 1/rms.  Two barriers.
template <int NTHR, int BAR, class ColFn>
__device__ __forceinline__ void rstd_finish(int ft, float s, int M, int MP, int h, float eps, FinSmem* fs, float* s_rstd, ColFn col) {
  const int TPT = NTHR / MP, width = TPT < 32 ? TPT : 32, nsub = TPT < 32 ? 1 : TPT / 32;
  for (int o = width >> 1; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if ((ft % width) == 0) fs->rpart[ft / width] = s;
  team_sync<NTHR, BAR>();
  if (ft < M && col(ft) >= 0) {
    float t = 0.f;
    for (int k = 0; k < nsub; ++k) t += fs->rpart[ft * nsub + k];
    s_rstd[ft] = 1.f / sqrtf(t / (float)h + eps);
  }
  team_sync<NTHR, BAR>();
}

// Piece sums of the group's tile(s) for the 8 tokens tok0 .. tok0+7, pieces in CTA order.  The thread ->
// element mapping follows the pieces' memory layout (coalesced), and the first four pieces of every
// element are requested before any is used.
template <int NTILE, int NTHR>
struct Gather {
  static constexpr int Q = NTILE * 1024 / NTHR;   // elements per thread (1024 elements per tile)
  float v[Q][4];
  __device__ __forceinline__ void issue(int ft, const GemmArgs& p, const GroupMeta* gm, int tok0, int MP) {
#pragma unroll
    for (int q = 0; q < Q; ++q) {
      const int e = ft + NTHR * q, row = (e >> 3) & 127;
      const int* m = gm->row[(e >> 10) * 8 + (row >> 4)];
      const float* src = p.part + (size_t)(row & 15) * MP + tok0 + (e & 7);
      const int n = m[0];
#pragma unroll
      for (int u = 0; u < 4; ++u) v[q][u] = u < n ? __ldcg(src + (size_t)m[1 + u] * 16 * MP) : 0.f;
    }
  }
  __device__ __forceinline__ void finish(int ft, const GemmArgs& p, const GroupMeta* gm, int tok0, int MP, FinSmem* fs) {
#pragma unroll
    for (int q = 0; q < Q; ++q) {
      const int e = ft + NTHR * q, row = (e >> 3) & 127;
      const int* m = gm->row[(e >> 10) * 8 + (row >> 4)];
      float acc = (((0.f + v[q][0]) + v[q][1]) + v[q][2]) + v[q][3];
      for (int u = 4; u < m[0]; ++u)  // rare: long reductions cut into many short ranges
        acc += __ldcg(p.part + ((size_t)m[1 + u] * 16 + (row & 15)) * MP + tok0 + (e & 7));
      fs->xs[e >> 10][row][e & 7] = acc;
    }
  }
};

// Sums v[0..NV) over the 128 rows of a tile (thread -> row = ft & 127, token class = ft >> 7); results valid
// in every thread; fixed order.  sh: NV floats per warp of the team (32 floats in all).
template <int NTHR, int BAR, int NV>
__device__ __forceinline__ void tile_rows_sum(int ft, float (&v)[NV], float* sh) {
  constexpr int NWARP = NTHR / 32;
  const int lane = ft & 31, warp = ft >> 5;
#pragma unroll
  for (int k = 0; k < NV; ++k) v[k] = warp_sum(v[k]);
  team_sync<NTHR, BAR>();
  if (lane == 0) {
#pragma unroll
    for (int k = 0; k < NV; ++k) sh[k * NWARP + warp] = v[k];
  }
  team_sync<NTHR, BAR>();
  const int c4 = (warp >> 2) * 4;  // warps c4 .. c4+3 hold the 128 rows of this token class
#pragma unroll
  for (int k = 0; k < NV; ++k) v[k] = sh[k * NWARP + c4] + sh[k * NWARP + c4 + 1] + sh[k * NWARP + c4 + 2] + sh[k * NWARP + c4 + 3];
}

// The fused epilogue of one completed group (one 128-row tile, or a pair of tiles).  It sits on the
// kernel's tail, so it is built around a single round trip to memory: every load it needs (pieces,
// residual, gain, sums of squares, RoPE entry) is requested up front, from addresses that depend on
// nothing loaded here (the piece table is already in shared memory); then come the reductions through
// shared memory and the stores.  s_pos[tok] = P_b + r (EPI_QKV), s_rstd preset to the <mask> rows' 1/rms.
// dry = true executes the same instructions without a single store to global memory (a measurement aid: a
// second call on the same group takes 3 us instead of 5.5, because the pieces, written by SMs all over the
// chip, are then close by - not because of the code: a dry pass ahead of time does not help).
// One instantiation per epilogue mode, so each mode only carries its own instructions; always inlined into the
// kernel, so that its many reads of the arguments are operands from the constant bank (out of line they were
// dependent loads through a pointer: about 2 us more on the tail of every projection).
template <int MODE, int NTHR, int BAR>
static __device__ __forceinline__ void finalize_group_t(int ft, const GemmArgs& p, int group, int MP, float* sh, float* s_rstd,
                                                     const int* s_pos, const GroupMeta* gm, FinSmem* fs, bool dry) {
  constexpr int NPAR = NTHR / 128;     // token classes: thread -> (row = ft & 127, class = ft >> 7)
  constexpr int NV = 8 / NPAR;         // tokens of an 8-token chunk per thread in the row-major modes
  constexpr int NP = 512 / NTHR;       // (token, pair) items per thread in EPI_QKV
  const EpiArgs& e = p.epi;
  const int M = p.s.M;
  const int Ta = group, Tb = group + p.pair_offset;
  const bool paired = p.pair_offset > 0;
  int s = 0;  // segment of tile Ta
  for (int i = 1; i < 6; ++i)
    if (i < p.s.nseg && Ta >= p.s.seg[i].tile0) s = i;
  const int row_base = (Ta - p.s.seg[s].tile0) * 128;       // first row of the tile inside its matrix
  const int rows_valid = min(128, p.s.seg[s].rows - row_base);
  const int row = ft & 127, par = ft >> 7;
  const int n = row_base + row;
  const int K = e.K;
  const auto col_id = [](int tok) { return tok; };
  const auto col_fresh = [K, &e](int tok) { return fresh_index(e, tok / K, tok % K); };
  constexpr bool rowmode = MODE == EPI_FC || MODE == EPI_RES;
  const int dh = e.dh, half = dh >> 1;
  const int pairs = MODE == EPI_QKV ? (rows_valid / dh) * half : 1;   // (head, i) pairs of this tile

  for (int tok0 = 0; tok0 < M; tok0 += 8) {
    // ---- every load, before any use
    Gather<2, NTHR> g2;
    Gather<1, NTHR> g1;
    if (paired) g2.issue(ft, p, gm, tok0, MP); else g1.issue(ft, p, gm, tok0, MP);
    unsigned short gam_raw = 0;
    if (rowmode && row < rows_valid) gam_raw = reinterpret_cast<const unsigned short*>(e.gamma)[n];
    float res[NV];
#pragma unroll
    for (int k = 0; k < NV; ++k) {
      res[k] = 0.f;
      const int t = tok0 + par + NPAR * k;
      if (MODE == EPI_RES && row < rows_valid && t < M) {
        // residual: the stream so far, or (first projection) g of a fresh row / the <mask> representation
        const int fi = e.res_in != nullptr ? -1 : fresh_index(e, t / K, t % K);
        const float* src = e.res_in != nullptr ? e.res_in + (size_t)t * e.h : (fi >= 0 ? e.res0 + (size_t)fi * e.h : e.mask_res);
        res[k] = __ldcg(src + n);
      }
    }
    float2 cs[NP];
#pragma unroll
    for (int k = 0; k < NP; ++k) {
      cs[k] = make_float2(1.f, 0.f);
      const int idx = ft + NTHR * k, ptok = tok0 + idx / pairs, pi = idx % pairs;
      if (MODE == EPI_QKV && s < 2 && idx < pairs * 8 && ptok < M)
        cs[k] = e.rope_tab[(size_t)s_pos[ptok] * half + (pi % half)];  // (cos, sin) of pos * theta^(-2i/d_h)
    }
    float rs = 0.f;
    if (tok0 == 0) {
      if (MODE == EPI_GATE_UP) rs = rstd_issue<NTHR>(ft, e.ss_in, e.ss_tiles, e.ss_mp, M, MP, col_id);
      if (MODE == EPI_QKV) rs = rstd_issue<NTHR>(ft, e.ss_in, e.ss_tiles, e.ss_mp, M, MP, col_fresh);
    }
    // ---- reductions through shared memory
    if (tok0 == 0) {
      if (MODE == EPI_GATE_UP) rstd_finish<NTHR, BAR>(ft, rs, M, MP, e.h, e.eps, fs, s_rstd, col_id);
      if (MODE == EPI_QKV) rstd_finish<NTHR, BAR>(ft, rs, M, MP, e.h, e.eps, fs, s_rstd, col_fresh);
    }
    if (paired) g2.finish(ft, p, gm, tok0, MP, fs); else g1.finish(ft, p, gm, tok0, MP, fs);
    team_sync<NTHR, BAR>();

    // ---- the mode's arithmetic and stores
    if (rowmode) {
      // FC: g = FC(features) on the fresh rows.  RES: x = residual + projection.  Both: residual stream,
      // gain-scaled hi/lo for the next projection, the tile's sum of squares for the next 1/rms.
      const float gam = __bfloat162float(__ushort_as_bfloat16(gam_raw));
      float x[NV], q[NV];
#pragma unroll
      for (int k = 0; k < NV; ++k) {
        const int t = tok0 + par + NPAR * k;
        x[k] = (row < rows_valid && t < M) ? res[k] + fs->xs[0][row][par + NPAR * k] : 0.f;
        q[k] = x[k] * x[k];
      }
      tile_rows_sum<NTHR, BAR, NV>(ft, q, sh);
      float* resw = MODE == EPI_FC ? e.res0 : e.res_out;
#pragma unroll
      for (int k = 0; k < NV; ++k) {
        const int t = tok0 + par + NPAR * k;
        // the FC's token index counts fresh rows only; its z row is the step's row (b, r)
        const int o = MODE == EPI_FC ? fresh_to_step_row(e, t < M ? t : 0) : t;
        if (row < rows_valid && t < M && !dry) {
          DART_CHECK(n < e.h && o >= 0 && o < e.B * e.K, e.status) {
            if (resw != nullptr) resw[(size_t)t * e.h + n] = x[k];
            bf16 hi, lo;
            split_bf16(x[k] * gam, hi, lo);
            e.out_hi[(size_t)o * e.ld_out + n] = hi;
            e.out_lo[(size_t)o * e.ld_out + n] = lo;
          }
        }
        if (row == 0 && t < M && !dry) e.ss_out[(size_t)Ta * MP + t] = q[k];
      }
    } else if (MODE == EPI_GATE_UP) {
      // u = SiLU(rstd * gate) * (rstd * up): the previous RMSNorm's 1/rms is applied here
#pragma unroll
      for (int k = 0; k < NV; ++k) {
        const int tl = par + NPAR * k, tok = tok0 + tl;
        if (row < rows_valid && tok < M && !dry) {
          const float gt = s_rstd[tok] * fs->xs[0][row][tl], up = s_rstd[tok] * fs->xs[1][row][tl];
          bf16 hi, lo;
          split_bf16(gt / (1.f + expf(-gt)) * up, hi, lo);
          DART_CHECK(n < e.ld_out && tok < e.B * e.K, e.status) {
            e.out_hi[(size_t)tok * e.ld_out + n] = hi;
            e.out_lo[(size_t)tok * e.ld_out + n] = lo;
          }
        }
      }
    } else if (MODE == EPI_QKV) {
      // y = rstd_g * (W[:, :h] z_g) + W[:, h:] z_e ; RoPE on q, k at position P_b + r ; q and the new rows'
      // k, v as hi/lo pairs ; the fresh rows' k, v appended to the cache.  segment 0,1,2 = q,k,v (g half);
      // the e half is the paired tile.
      const int kind = s;
#pragma unroll
      for (int k = 0; k < NP; ++k) {
        const int idx = ft + NTHR * k, ptok = tok0 + idx / pairs, pi = idx % pairs;
        if (idx < pairs * 8 && ptok < M && !dry) {
          const int tl = ptok - tok0, tok = ptok;
          const int hl = pi / half, i = pi - hl * half;
          const int ra = hl * dh + i, rb = ra + half;
          const float x1 = s_rstd[tok] * fs->xs[0][ra][tl] + fs->xs[1][ra][tl];
          const float x2 = s_rstd[tok] * fs->xs[0][rb][tl] + fs->xs[1][rb][tl];
          const int b = tok / K, r = tok % K;
          float o1 = x1, o2 = x2;
          if (kind < 2) {
            o1 = x1 * cs[k].x - x2 * cs[k].y;
            o2 = x2 * cs[k].x + x1 * cs[k].y;
          }
          bf16 h1, l1, h2, l2;
          split_bf16(o1, h1, l1);
          split_bf16(o2, h2, l2);
          const int head = (row_base / dh) + hl;
          if (kind == 0) {
            const size_t o = (((size_t)b * e.Hq + head) * K + r) * dh;
            DART_CHECK(head < e.Hq && b < e.B, e.status) {
              e.q_hi[o + i] = h1; e.q_hi[o + i + half] = h2;
              e.q_lo[o + i] = l1; e.q_lo[o + i + half] = l2;
            }
          } else {
            bf16* side = (kind == 1 ? e.k_new : e.v_new) + ((size_t)b * e.Hkv + head) * 16 * dh;
            side[(size_t)r * dh + i] = h1; side[(size_t)r * dh + i + half] = h2;
            side[(size_t)(8 + r) * dh + i] = l1; side[(size_t)(8 + r) * dh + i + half] = l2;
            if (fresh_index(e, b, r) >= 0) {
              bf16* dst = (kind == 1 ? e.k_cache : e.v_cache) + (((size_t)b * e.Hkv + head) * e.P_cap + s_pos[tok]) * dh;
              DART_CHECK(s_pos[tok] >= 0 && s_pos[tok] < e.P_cap && head < e.Hkv, e.status) {   // the append stays inside the sequence's cache rows
                dst[i] = h1;
                dst[i + half] = h2;
              }
            }
          }
        }
      }
    }
    team_sync<NTHR, BAR>();
  }
}

template <int NTHR, int BAR>
static __device__ __forceinline__ void finalize_group(int ft, const GemmArgs& p, int group, int MP, float* sh, float* s_rstd,
                                                      const int* s_pos, const GroupMeta* gm, FinSmem* fs, bool dry = false) {
  switch (p.epi.mode) {
    case EPI_FC: finalize_group_t<EPI_FC, NTHR, BAR>(ft, p, group, MP, sh, s_rstd, s_pos, gm, fs, dry); break;
    case EPI_QKV: finalize_group_t<EPI_QKV, NTHR, BAR>(ft, p, group, MP, sh, s_rstd, s_pos, gm, fs, dry); break;
    case EPI_RES: finalize_group_t<EPI_RES, NTHR, BAR>(ft, p, group, MP, sh, s_rstd, s_pos, gm, fs, dry); break;
    default: finalize_group_t<EPI_GATE_UP, NTHR, BAR>(ft, p, group, MP, sh, s_rstd, s_pos, gm, fs, dry); break;
  }
}

// Shifted token embedding of the fresh rows (Section 3.2): e = E[token], normalised (its 1/rms needs nothing
// else) and written as the second half of the fresh row's z.  Runs on a team of NTHR threads that synchronises on
// named barrier BAR (warps that idle while the projection streams), with the arguments read from the kernel's
// constant bank.  red: NTHR / 32 floats of shared memory.
template <int NTHR, int BAR>
static __device__ __forceinline__ void embed_row_team(const EpiArgs& e, int ft, float* red, int ftok) {
  const int orow = fresh_to_step_row(e, ftok);
  const int id = min(max(e.tokens[ftok], 0), e.vocab - 1);
  const int h = e.h;
  const bf16* row = e.embed + (size_t)id * h;
  float ss = 0.f;
  for (int n = ft; n < h; n += NTHR) {
    const float v = __bfloat162float(row[n]);
    ss += v * v;
  }
  ss = warp_sum(ss);
  if ((ft & 31) == 0) red[ft >> 5] = ss;
  team_sync<NTHR, BAR>();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < NTHR / 32; ++w) tot += red[w];
  const float rs = 1.f / sqrtf(tot / (float)h + e.eps);
  bf16* out_hi = e.out_hi + (size_t)orow * e.ld_out + h;
  bf16* out_lo = e.out_lo + (size_t)orow * e.ld_out + h;
  const bf16* gam = e.gamma_e;
  for (int n = ft; n < h; n += NTHR) {
    bf16 hi, lo;
    split_bf16(__bfloat162float(row[n]) * rs * __bfloat162float(gam[n]), hi, lo);
    out_hi[n] = hi;
    out_lo[n] = lo;
  }
  team_sync<NTHR, BAR>();   // red is free for the next row
}

}  // namespace dart
