// Weight-streaming small-M GEMM ("rows" mode) for the draft layer's projections
// (FC, QKV, o_proj, gate/up, down -- Section 3.2's single decoder layer).
//
// The op is HBM-bound: M = batch*K token rows (8..128) against weight matrices of 10^7..10^8
// elements, i.e. M flop per weight byte.  Design:
//   * weights are the MMA's M-side operand (16 weight rows x 16 k per mma.sync.m16n8k16),
//     token rows are the 8-wide N side, so M = 8 tokens is an exact fit;
//   * weight fragments go global -> registers with 128-bit coalesced loads, each quad reading
//     64 contiguous bytes (two whole sectors) of a weight row per instruction and one full
//     128-byte line per k-step; the k index is permuted identically on both operands so that
//     the 2 x 16 bytes a thread loads are exactly its fragment slots;
//   * activations (a few hundred KB, bf16 hi + lo) are read through L1 by every warp;
//   * the flattened (128-row tile, k-step) space is cut into gridDim.x equal ranges, so every
//     CTA streams the same number of bytes (no tail wave); per-tile partials are summed in CTA
//     order by the finalize kernel that follows (deterministic, no atomics).
#include "common.cuh"
#include "kernels.h"

namespace dart {

struct GemmRowsArgs {
  GemmSeg seg[3];
  int nseg;
  int Kd, SK, slots;
  long long U;
  const bf16* x_hi;
  const bf16* x_lo;
  long long ldx;
  int M;
  float* part;
};

struct RowCursor {
  int tile, ks;
  const bf16* r0;
  const bf16* r1;
  bool valid;
  __device__ __forceinline__ void set_tile(const GemmRowsArgs& p, int warp, int g) {
    int s = 0;
    if (p.nseg > 1 && tile >= p.seg[1].tile0) s = 1;
    if (p.nseg > 2 && tile >= p.seg[2].tile0) s = 2;
    const int row0 = (tile - p.seg[s].tile0) * 128 + warp * 16;
    valid = row0 < p.seg[s].rows;
    r0 = p.seg[s].W + (size_t)(valid ? row0 + g : 0) * p.Kd;
    r1 = r0 + (size_t)(valid ? 8 : 0) * p.Kd;
  }
  __device__ __forceinline__ void advance(const GemmRowsArgs& p, int warp, int g) {
    if (++ks == p.SK) {
      ks = 0;
      ++tile;
      set_tile(p, warp, g);
    }
  }
};

// FULL: Kd is a multiple of 64, every segment's rows a multiple of 128 and all MP token rows are
// valid, so the streaming loop carries no bounds predicates.
template <int NT, bool HAS_LO, int PF, bool FULL>
__global__ void __launch_bounds__(256, (NT <= 4 ? 2 : 1)) gemm_rows_kernel(const GemmRowsArgs p) {
  constexpr int MP = 8 * NT;
  const int c = blockIdx.x, G = gridDim.x;
  const long long u0 = ((long long)c * p.U) / G, u1 = ((long long)(c + 1) * p.U) / G;
  if (u0 >= u1) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int tile_first = (int)(u0 / p.SK);

  float acc[NT][4];
#pragma unroll
  for (int n = 0; n < NT; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
  uint4 a[PF][4];

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
          const bf16* xp = p.x_hi + (size_t)tok * p.ldx;
          const bf16* xq = p.x_lo + (size_t)tok * p.ldx;
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
          const uint32_t xh[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
          const uint32_t xl[8] = {l0.x, l0.y, l0.z, l0.w, l1.x, l1.y, l1.z, l1.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            mma_bf16_16816(acc[n], w0[2 * j], w1[2 * j], w0[2 * j + 1], w1[2 * j + 1], xh[2 * j], xh[2 * j + 1]);
            if (HAS_LO)
              mma_bf16_16816(acc[n], w0[2 * j], w1[2 * j], w0[2 * j + 1], w1[2 * j + 1], xl[2 * j], xl[2 * j + 1]);
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
        }
        cp.advance(p, warp, g);
      }
    }
  }
}

template <int NT, bool HAS_LO, int PF>
static cudaError_t launch_t(const GemmRowsArgs& a, int grid, bool full, cudaStream_t st) {
  if (full)
    gemm_rows_kernel<NT, HAS_LO, PF, true><<<grid, 256, 0, st>>>(a);
  else
    gemm_rows_kernel<NT, HAS_LO, PF, false><<<grid, 256, 0, st>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_gemm_rows(const GemmPlan& plan, const bf16* x_hi, const bf16* x_lo, long long ldx, int M,
                             float* part, cudaStream_t st) {
  GemmRowsArgs a;
  for (int i = 0; i < 3; ++i) a.seg[i] = plan.seg[i < plan.nseg ? i : 0];
  a.nseg = plan.nseg;
  a.Kd = plan.Kd; a.SK = plan.SK; a.slots = plan.slots; a.U = plan.U;
  a.x_hi = x_hi; a.x_lo = x_lo; a.ldx = ldx; a.M = M; a.part = part;
  const int MP = padded_tokens(M);
  const bool lo = x_lo != nullptr;
  bool full = (plan.Kd % 64 == 0) && (M == MP);
  for (int i = 0; i < plan.nseg; ++i) full = full && (plan.seg[i].rows % 128 == 0);
  if (MP == 8) return lo ? launch_t<1, true, 4>(a, plan.grid, full, st) : launch_t<1, false, 4>(a, plan.grid, full, st);
  if (MP == 32) return lo ? launch_t<4, true, 2>(a, plan.grid, full, st) : launch_t<4, false, 2>(a, plan.grid, full, st);
  return lo ? launch_t<16, true, 2>(a, plan.grid, full, st) : launch_t<16, false, 2>(a, plan.grid, full, st);
}

}  // namespace dart
