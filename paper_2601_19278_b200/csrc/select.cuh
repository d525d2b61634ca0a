// Selection helpers shared by the tree builder and the top-k merge: candidates as 64-bit keys, warp-level
// bitonic sort, and a block-wide "best 64" merge tree that lives in registers.
#pragma once
#include "common.cuh"

namespace dart {

// A candidate as one 64-bit key whose unsigned order is the total order (score desc, index asc):
// high word = the score's bits mapped so that larger floats give larger integers (-0 is first folded
// into +0, so that equal scores compare equal), low word = ~index.  The larger key precedes.
typedef unsigned long long Key;
constexpr Key kPadKey = 0ull;  // below every real key: (-inf score would map above 0; index bits of a pad are 0)

__device__ __forceinline__ Key make_key(float s, int c) {
  uint32_t u = __float_as_uint(s + 0.0f);
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  return ((Key)u << 32) | (Key)(~(uint32_t)c);
}
__device__ __forceinline__ int key_index(Key k) { return (int)(~(uint32_t)k); }
__device__ __forceinline__ Key shfl_key(Key k, int src) { return __shfl_sync(0xffffffffu, k, src); }
__device__ __forceinline__ Key kmax(Key a, Key b) { return a > b ? a : b; }
__device__ __forceinline__ Key kmin(Key a, Key b) { return a > b ? b : a; }

// Sort one key per lane so that lane 0 holds the largest.
__device__ __forceinline__ void warp_sort(Key& x, int lane) {
#pragma unroll
  for (int k = 2; k <= 32; k <<= 1) {
#pragma unroll
    for (int j = k >> 1; j > 0; j >>= 1) {
      const Key o = shfl_key(x, lane ^ j);
      const bool up = (lane & k) == 0, lower = (lane & j) == 0;
      x = (lower == up) ? kmax(x, o) : kmin(x, o);
    }
  }
}

// (x0, x1) hold a bitonic sequence of 64 keys (position p = 32*reg + lane); sort it, largest first.
__device__ __forceinline__ void bitonic_merge64(Key& x0, Key& x1, int lane) {
  const Key hi = kmax(x0, x1), lo = kmin(x0, x1);
  x0 = hi;
  x1 = lo;
#pragma unroll
  for (int j = 16; j > 0; j >>= 1) {
    const bool lower = (lane & j) == 0;
    const Key o0 = shfl_key(x0, lane ^ j), o1 = shfl_key(x1, lane ^ j);
    x0 = lower ? kmax(x0, o0) : kmin(x0, o0);
    x1 = lower ? kmax(x1, o1) : kmin(x1, o1);
  }
}

// Merge the sorted 64-key run (y0, y1) of the same warp into (x0, x1), keeping the best 64 sorted.
__device__ __forceinline__ void merge_keep64(Key& x0, Key& x1, Key y0, Key y1, int lane) {
  const Key r0 = shfl_key(y1, 31 - lane), r1 = shfl_key(y0, 31 - lane);  // y reversed: y[63 - p]
  x0 = kmax(x0, r0);
  x1 = kmax(x1, r1);
  bitonic_merge64(x0, x1, lane);
}

// Best 64 of the block's candidates (one key per thread; pads are kPadKey), sorted, in warp 0's (x0, x1).
// xk: shared scratch of 64 keys per warp.  `pred` is OR-reduced over the block in the first barrier and returned.  nruns = warps that hold
// candidates.  All threads of the block must call this.
__device__ __forceinline__ int block_best64(Key key, int nruns, Key* xk, int pred, Key& x0, Key& x1) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  warp_sort(key, lane);
  x0 = key;
  x1 = kPadKey;
  int any = 0;
  bool first = true;
  for (int stride = 1; stride < nruns || first; stride <<= 1) {
    const bool donor = (warp & (2 * stride - 1)) == stride && warp < nruns;
    if (donor) {
      xk[warp * 64 + lane] = x0;
      xk[warp * 64 + 32 + lane] = x1;
    }
    if (first) { any = __syncthreads_or(pred); first = false; } else __syncthreads();
    if ((warp & (2 * stride - 1)) == 0 && warp + stride < nruns) {
      const int pw = (warp + stride) * 64;
      x0 = kmax(x0, xk[pw + 63 - lane]);
      x1 = kmax(x1, xk[pw + 31 - lane]);
      bitonic_merge64(x0, x1, lane);
    }
  }
  return any;
}

}  // namespace dart
