// Shared weight-streaming core of the projections and the LM head.
//
// Work unit = (16-row tile "m-tile", k-round), a k-round being NW consecutive 64-wide k-steps, one per
// warp: the NW warps of a CTA read NW * 128 contiguous bytes of each of the m-tile's 16 rows at the same
// time, then move on along the row.  On B200 this pattern streams at ~6.8 TB/s with 32 warps per SM and
// only one or two k-steps of loads in flight per warp (measured with a load-only kernel; one warp per 16
// rows tops out near 5.8 TB/s, 16 warps per SM near 5.3 TB/s), so the kernels run 2 CTAs x 16 warps per
// SM with at most 64 registers per thread.
//
// Each warp multiplies its k-slices on mma.sync.m16n8k16 (weights = the M side, 8 token rows = the N
// side, bf16 hi + lo activations as two MMAs into one fp32 accumulator).  When an m-tile (or the CTA's
// share of it) is done, the warps' partial tiles are written to shared memory and the caller's functor
// sums and consumes them.
#pragma once
#include "common.cuh"
#include "kernels.h"

namespace dart {

// Position of one warp in the unit sequence.
struct UnitCursor {
  int mt;       // global m-tile index (128-row tile * 8 + sub-tile)
  int kr;       // k-round inside the m-tile
  const bf16* w0;  // row g of the m-tile, at this warp's k-step of round kr
  int ldw;      // row stride of the segment's matrix
  int xoff;     // activation column offset of the segment
  bool valid;   // the m-tile lies inside its matrix
  __device__ __forceinline__ void seek(const StreamArgs& a, int mt_, int kr_, int warp, int g, int NW) {
    mt = mt_;
    kr = kr_;
    const int tile = mt >> 3;
    int s = 0;
#pragma unroll
    for (int i = 1; i < 6; ++i)
      if (i < a.nseg && tile >= a.seg[i].tile0) s = i;
    const int row0 = (mt - a.seg[s].tile0 * 8) * 16;
    valid = row0 < a.seg[s].rows;
    w0 = a.seg[s].W + (size_t)(valid ? row0 + g : 0) * a.seg[s].ld + (size_t)(kr * NW + warp) * 64;
    ldw = a.seg[s].ld;
    xoff = a.seg[s].xoff;
  }
};

// Streams units [u0, u1) of the flattened (m-tile, k-round) space.  `epi.after_wait()` is called by every
// thread once the predecessor kernel has completed (it may contain CTA-wide barriers).  `epi.mtile_done(mt, buf, last)` is
// called by every thread of the CTA after the partial tiles of m-tile `mt` have been written to
// red[buf] = [NW][16 rows][MP tokens] (RB buffers) and a __syncthreads(); it may contain further CTA-wide barriers.
// FULL: Kd is a multiple of 64*NW, every m-tile is valid and all MP token rows exist.
template <int NT, bool HAS_LO, int PF, int NW, int RB, bool FULL, class Epi>
__device__ __forceinline__ void stream_units(const StreamArgs& a, long long u0, long long u1, float* red, Epi& epi) {
  constexpr int MP = 8 * NT;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int c0 = chunk_k0(t), c1 = chunk_k1(t);
  const int n = (int)(u1 - u0);

  // activation row of each token this thread feeds to the MMA (token i*8+g)
  const bf16* xh[NT];
  const long long xlo_delta = a.x_lo - a.x_hi;
#pragma unroll
  for (int i = 0; i < NT; ++i) {
    int tok = i * 8 + g;
    if (tok >= a.M) tok = 0;  // padded token rows read row 0; their results are never used
    xh[i] = a.x_hi + (long long)tok * a.ldx;
  }

  float acc[NT][4];
#pragma unroll
  for (int i = 0; i < NT; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
  uint4 wreg[PF][4];

  UnitCursor ld, cp;
  ld.seek(a, (int)(u0 / a.KR), (int)(u0 % a.KR), warp, g, NW);
  cp = ld;
  auto advance = [&](UnitCursor& c) {
    if (c.kr + 1 < a.KR) {
      ++c.kr;
      c.w0 += 64 * NW;
    } else {
      c.seek(a, c.mt + 1, 0, warp, g, NW);
    }
  };
  auto issue = [&](uint4(&dst)[4]) {
    const bf16* r0 = ld.w0;
    const bf16* r1 = r0 + (size_t)8 * ld.ldw;
    if (FULL) {
      dst[0] = ld_stream16(r0 + c0);
      dst[1] = ld_stream16(r0 + c1);
      dst[2] = ld_stream16(r1 + c0);
      dst[3] = ld_stream16(r1 + c1);
    } else {
      const int k = (ld.kr * NW + warp) * 64;
      const bool va = ld.valid && k + c0 < a.Kd, vb = ld.valid && k + c1 < a.Kd;
      const uint4 z = make_uint4(0, 0, 0, 0);
      dst[0] = va ? ld_stream16(r0 + c0) : z;
      dst[1] = vb ? ld_stream16(r0 + c1) : z;
      dst[2] = va ? ld_stream16(r1 + c0) : z;
      dst[3] = vb ? ld_stream16(r1 + c1) : z;
    }
    advance(ld);
  };

#pragma unroll
  for (int s = 0; s < PF; ++s)
    if (s < n) issue(wreg[s]);
  // the weights above depend on no earlier kernel; everything below (activations, partials) does
  pdl_wait();
  epi.after_wait();

  int buf = 0;
  for (int u = 0; u < n; u += PF) {
#pragma unroll
    for (int s = 0; s < PF; ++s) {
      if (u + s < n) {
        const int k = (cp.kr * NW + warp) * 64;
        const uint32_t w0[8] = {wreg[s][0].x, wreg[s][0].y, wreg[s][0].z, wreg[s][0].w,
                                wreg[s][1].x, wreg[s][1].y, wreg[s][1].z, wreg[s][1].w};
        const uint32_t w1[8] = {wreg[s][2].x, wreg[s][2].y, wreg[s][2].z, wreg[s][2].w,
                                wreg[s][3].x, wreg[s][3].y, wreg[s][3].z, wreg[s][3].w};
#pragma unroll
        for (int i = 0; i < NT; ++i) {
          uint4 h0 = make_uint4(0, 0, 0, 0), h1 = h0, l0 = h0, l1 = h0;
          const bf16* xp = xh[i] + cp.xoff + k;
          const bf16* xq = xp + xlo_delta;
          if (FULL) {
            h0 = ld_act16(xp + c0);
            h1 = ld_act16(xp + c1);
            if (HAS_LO) { l0 = ld_act16(xq + c0); l1 = ld_act16(xq + c1); }
          } else {
            if (k + c0 < a.Kd) {
              h0 = ld_act16(xp + c0);
              if (HAS_LO) l0 = ld_act16(xq + c0);
            }
            if (k + c1 < a.Kd) {
              h1 = ld_act16(xp + c1);
              if (HAS_LO) l1 = ld_act16(xq + c1);
            }
          }
          const uint32_t xhv[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
          const uint32_t xlv[8] = {l0.x, l0.y, l0.z, l0.w, l1.x, l1.y, l1.z, l1.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            mma_bf16_16816(acc[i], w0[2 * j], w1[2 * j], w0[2 * j + 1], w1[2 * j + 1], xhv[2 * j], xhv[2 * j + 1]);
            if (HAS_LO)
              mma_bf16_16816(acc[i], w0[2 * j], w1[2 * j], w0[2 * j + 1], w1[2 * j + 1], xlv[2 * j], xlv[2 * j + 1]);
          }
        }
        if (u + s + PF < n) issue(wreg[s]);

        const bool last = (u + s == n - 1);
        if (cp.kr == a.KR - 1 || last) {
          // the CTA's share of this m-tile is complete: hand the NW partial tiles to the epilogue
          float* rw = red + ((size_t)buf * NW + warp) * 16 * MP;
#pragma unroll
          for (int i = 0; i < NT; ++i) {
            *reinterpret_cast<float2*>(rw + g * MP + i * 8 + 2 * t) = make_float2(acc[i][0], acc[i][1]);
            *reinterpret_cast<float2*>(rw + (g + 8) * MP + i * 8 + 2 * t) = make_float2(acc[i][2], acc[i][3]);
            acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
          }
          __syncthreads();
          epi.mtile_done(cp.mt, buf, last);
          if (RB == 1) __syncthreads(); else buf ^= 1;
        }
        advance(cp);
      }
    }
  }
}

// Sum of the NW partial tiles for element (row, tok) of red[buf].
template <int NW, int MP>
__device__ __forceinline__ float red_sum(const float* red, int buf, int row, int tok) {
  float v = 0.f;
#pragma unroll
  for (int w = 0; w < NW; ++w) v += red[((size_t)buf * NW + w) * 16 * MP + row * MP + tok];
  return v;
}

}  // namespace dart
