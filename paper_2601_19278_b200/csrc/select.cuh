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

// ------------------------------------------------------------------------------------------------------
// Best 64 of the block's candidates by a value histogram (the tree builder's per-level selection).
//
// The merge tree above costs a 15-stage warp sort and log2(warps) merge rounds with a block barrier each.  This
// routine reaches the same result -- the 64 largest keys of the block in order -- in four barriers and no sort:
//   1. block-wide minimum and maximum of the (finite) scores;
//   2. a 256-bin histogram of the scores between them (bin 0 = the maximum; the map score -> bin is monotone);
//   3. every warp scans the histogram for the first bin b* at which the running count reaches 64: the 64 largest
//      keys all lie in bins <= b*; the candidates of those bins (a few more than 64, unless many scores coincide)
//      are appended to a list;
//   4. every survivor counts the survivors that precede it -- its rank, because nothing outside the list precedes
//      a survivor of rank < 64 -- and stores its key at that position.
// Keys are unique, so the result does not depend on the order in which threads append.  Many equal or nearly
// equal scores only make step 4 longer (the list is as long as the block at worst), never wrong.
// ------------------------------------------------------------------------------------------------------
constexpr int kSelectCap = 1024;   // candidates per block (one per thread)
struct SelectSmem {
  unsigned umax, umin;   // order-preserving images of the largest and smallest finite score (reset by every call for the next)
  int cnt;
  int pad;
  int hist[256];
  Key surv[kSelectCap + 16];
};

// Order-preserving image of a float: larger floats give larger integers (-0 counts as +0).
__device__ __forceinline__ uint32_t float_order(float s) {
  const uint32_t u = __float_as_uint(s + 0.0f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float float_unorder(uint32_t u) { return __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u); }

// Once per kernel, before the first block_select64 (followed by a barrier).
__device__ __forceinline__ void block_select_init(SelectSmem* ss) {
  if (threadIdx.x == 0) { ss->umax = 0u; ss->umin = 0xffffffffu; }
}

#ifdef DART_TREE_TL
__device__ long long g_sel_tl[8];
#define SEL_STAMP(i) do { if (threadIdx.x == 0) g_sel_tl[i] = clock64() - sel_t0; } while (0)
#else
#define SEL_STAMP(i) do {} while (0)
#endif
// key: the thread's candidate (kPadKey: none), made from `score`.  emit(r, key, any) is called exactly once for every
// r in 0 .. 63, by some thread, before the routine's last barrier: key = the r-th best of the block (kPadKey past the
// last candidate), any = the OR of `pred` over the block, which is also returned.  after1() runs in every thread right
// after the first barrier (the caller's earlier shared-memory reads are complete by then), during3() after the thread's
// part of step 4.  All threads must call; four barriers.
template <class Emit, class F1, class F3>
__device__ __forceinline__ int block_select64(Key key, float score, int pred, SelectSmem* ss, Emit&& emit, F1&& after1, F3&& during3) {
  const int tid = threadIdx.x, lane = tid & 31, nthr = blockDim.x;
#ifdef DART_TREE_TL
  const long long sel_t0 = clock64();
#endif
  const bool valid = key != kPadKey;
  const bool fin = valid && fabsf(score) <= 3.0e38f;
  const uint32_t uo = float_order(score);
  const uint32_t wmx = __reduce_max_sync(0xffffffffu, fin ? uo : 0u), wmn = __reduce_min_sync(0xffffffffu, fin ? uo : 0xffffffffu);
  if (lane == 0 && wmx != 0u) { atomicMax(&ss->umax, wmx); atomicMin(&ss->umin, wmn); }
  for (int e = tid; e < 256; e += nthr) ss->hist[e] = 0;
  for (int e = tid; e < kSelectCap + 16; e += nthr) ss->surv[e] = kPadKey;   // pads never precede anything: the rank loop needs no tail
  if (tid == 0) ss->cnt = 0;
  SEL_STAMP(0);
  const int any = __syncthreads_or(pred);                                   // ---- barrier 1
  SEL_STAMP(1);
  after1();
  const uint32_t umx = ss->umax, umn = ss->umin;
  const float mx = float_unorder(umx), mn = float_unorder(umn);
  const float scale = (umx > umn && umx != 0u) ? 255.f / (mx - mn) : 0.f;
  int bin = 255;
  if (fin) {
    const float d = (mx - score) * scale;        // monotone in the score: a larger score never gets a larger bin
    bin = d < 255.f ? (int)d : 255;
  }
  if (valid) atomicAdd(&ss->hist[bin], 1);
  SEL_STAMP(2);
  __syncthreads();                                                          // ---- barrier 2
  SEL_STAMP(3);
  int pre[8];   // running count within this lane's eight bins
  {
    const int4 a = reinterpret_cast<const int4*>(ss->hist)[lane * 2], b = reinterpret_cast<const int4*>(ss->hist)[lane * 2 + 1];
    pre[0] = a.x; pre[1] = pre[0] + a.y; pre[2] = pre[1] + a.z; pre[3] = pre[2] + a.w;
    pre[4] = pre[3] + b.x; pre[5] = pre[4] + b.y; pre[6] = pre[5] + b.z; pre[7] = pre[6] + b.w;
  }
  int cum = pre[7];
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, cum, o);
    if (lane >= o) cum += v;
  }
  const int total = __shfl_sync(0xffffffffu, cum, 31);
  const int target = total < 64 ? total : 64;
  const unsigned reach = __ballot_sync(0xffffffffu, cum >= target);        // never empty: lane 31 holds the total
  const int l0 = __ffs(reach) - 1;
  int bstar = lane * 8 + 7;
  {
    const int before = cum - pre[7];
#pragma unroll
    for (int q = 6; q >= 0; --q)
      if (before + pre[q] >= target) bstar = lane * 8 + q;   // scanning down keeps the first bin that reaches the target
  }
  bstar = __shfl_sync(0xffffffffu, bstar, l0);
  {
    // the candidates of bins <= b* are appended to the list, one atomic per warp
    const bool keep = valid && bin <= bstar;
    const unsigned km = __ballot_sync(0xffffffffu, keep);
    int basep = 0;
    if (km != 0u) {
      if (lane == __ffs(km) - 1) basep = atomicAdd(&ss->cnt, __popc(km));
      basep = __shfl_sync(0xffffffffu, basep, __ffs(km) - 1);
      if (keep) ss->surv[basep + __popc(km & ((1u << lane) - 1u))] = key;
    }
  }
  if (tid == 0) { ss->umax = 0u; ss->umin = 0xffffffffu; }   // for the next call (this call's readers are past barrier 2)
  SEL_STAMP(4);
  __syncthreads();                                                          // ---- barrier 3
  SEL_STAMP(5);
  const int c = ss->cnt;
  {
    // rank of a survivor = the survivors that precede it; P threads (adjacent lanes) share one survivor's count
    int P = 1;
    while (P < 8 && c * P * 2 <= nthr) P <<= 1;
    const int sv = tid / P, part = tid & (P - 1);
    const Key me = sv < c ? ss->surv[sv] : ~0ull;
    int r = 0;
    const ulonglong2* pairs = reinterpret_cast<const ulonglong2*>(ss->surv);
    const int npair = (c + 1) >> 1;
    for (int o = part; o < npair; o += P) {
      const ulonglong2 q = pairs[o];
      r += (q.x > me ? 1 : 0) + (q.y > me ? 1 : 0);
    }
    for (int o = 1; o < P; o <<= 1) r += __shfl_xor_sync(0xffffffffu, r, o);
    if (sv < c && part == 0 && r < 64) emit(r, me, any);
  }
  for (int e = tid; e < 64; e += nthr)
    if (e >= c) emit(e, kPadKey, any);              // fewer than 64 candidates in all: the rest are pads
  SEL_STAMP(6);
  during3();
  __syncthreads();                                                          // ---- barrier 4
#ifdef DART_TREE_TL
  if (threadIdx.x == 0) g_sel_tl[7] = c;
#endif
  return any;
}

}  // namespace dart
