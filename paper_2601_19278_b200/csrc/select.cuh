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
// routine reaches the same result -- the 64 largest keys of the block in order -- without a sort:
//   0. block-wide minimum and maximum of the (finite) scores (one warp reduction instruction each);
//   1. a 64-bin histogram of the scores between them (bin 0 = the maximum; the map score -> bin is monotone);
//   2. every warp scans the histogram for the first bin b* at which the running count reaches 64: the 64 largest
//      keys all lie in bins <= b* (a few more than 64 candidates, unless many scores coincide);
//   3. those survivors are packed into a list, warp after warp (offsets from the warps' counts);
//   4. every survivor counts the survivors that precede it -- its rank, because nothing outside the list precedes
//      a survivor of rank < 64 -- and reports its key with that rank.
// Keys are unique, so ranks do not depend on the order of the list.  Many equal or nearly equal scores only make
// step 4 longer (the list is as long as the block at worst), never wrong.  Measured on B200 with 17 warps resident:
// a shared-memory atomic that returns a value costs ~150 cycles and same-address lanes of a warp take turns at that
// price, a block barrier ~50, an integer division ~140 -- so there is none of the first and the last here, and every
// instruction that all warps execute costs four issue cycles.
// ------------------------------------------------------------------------------------------------------
constexpr int kSelectCap = 1024;   // candidates per block (one per thread)
struct SelectSmem {
  unsigned red_max[32], red_min[32];   // per warp: order-preserving images of its largest and smallest finite score
  int hist[64];
  int wcount[32];                      // per warp: its survivors
  Key surv[kSelectCap + 2];
};

// Order-preserving image of a float: larger floats give larger integers (-0 counts as +0).
__device__ __forceinline__ uint32_t float_order(float s) {
  const uint32_t u = __float_as_uint(s + 0.0f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float float_unorder(uint32_t u) { return __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u); }

// Once per kernel, before the first block_select64 (followed by a barrier).
__device__ __forceinline__ void block_select_init(SelectSmem* ss) {
  if (threadIdx.x < 64) ss->hist[threadIdx.x] = 0;
}

#ifdef DART_TREE_TL
__device__ long long g_sel_tl[12];
#define SEL_STAMP(i) do { if (threadIdx.x == 0) g_sel_tl[i] = clock64() - sel_t0; } while (0)
#else
#define SEL_STAMP(i) do {} while (0)
#endif
// key: the thread's candidate (kPadKey: none), made from `score`.  emit(r, key, any) is called exactly once for every
// r in 0 .. 63, by some thread, before the routine's last barrier: key = the r-th best of the block (kPadKey past the
// last candidate), any = the OR of `pred` over the block, which is also returned.  after1() runs in every thread right
// after the first barrier (the caller's earlier shared-memory reads are complete by then), during4() after the thread's
// part of step 4.  A warp whose threads all pass idle = true (and no candidates) only takes part in the first and the
// last barrier: the caller may give it other work in after1(), which then runs beside steps 1 to 4 of the others.
// n_active: threads that pass idle = false (a multiple of 32, at least 64).  All threads must call.
template <class Emit, class F1, class F4>
__device__ __forceinline__ int block_select64(Key key, float score, int pred, bool idle, int n_active, SelectSmem* ss, Emit&& emit,
                                              F1&& after1, F4&& during4) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarp = blockDim.x >> 5;
#ifdef DART_TREE_TL
  const long long sel_t0 = clock64();
#endif
  const bool valid = key != kPadKey;
  const bool fin = valid && fabsf(score) <= 3.0e38f;
  {
    const uint32_t uo = float_order(score);
    const uint32_t wmx = __reduce_max_sync(0xffffffffu, fin ? uo : 0u), wmn = __reduce_min_sync(0xffffffffu, fin ? uo : 0xffffffffu);
    if (lane == 0) { ss->red_max[warp] = wmx; ss->red_min[warp] = wmn; }
  }
  SEL_STAMP(0);
  const int any = __syncthreads_or(pred);                                   // ---- barrier 0
  SEL_STAMP(1);
  after1();
  if (!idle) {
    // ---- step 1
    int bin = 63;
    {
      const uint32_t umx = __reduce_max_sync(0xffffffffu, lane < nwarp ? ss->red_max[lane] : 0u);
      const uint32_t umn = __reduce_min_sync(0xffffffffu, lane < nwarp ? ss->red_min[lane] : 0xffffffffu);
      const float mx = float_unorder(umx), mn = float_unorder(umn);
      const float scale = (umx > umn && umx != 0u) ? __fdividef(63.f, mx - mn) : 0.f;
      if (fin) {
        const float d = (mx - score) * scale;        // monotone in the score: a larger score never gets a larger bin
        bin = d < 63.f ? (int)d : 63;
      }
      if (valid) atomicAdd(&ss->hist[bin], 1);       // no result needed (grouping equal bins with match.any first was slower)
    }
    SEL_STAMP(2);
    asm volatile("bar.sync 1, %0;" ::"r"(n_active) : "memory");             // ---- barrier 1
    SEL_STAMP(3);
    // ---- step 2: every warp scans the histogram
    int c, local;
    bool keep;
    {
      const int2 h = reinterpret_cast<const int2*>(ss->hist)[lane];
      int cum = h.x + h.y;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, cum, o);
        if (lane >= o) cum += v;
      }
      const int total = __shfl_sync(0xffffffffu, cum, 31);
      const int target = total < 64 ? total : 64;
      const int l0 = __ffs(__ballot_sync(0xffffffffu, cum >= target)) - 1;   // never empty: lane 31 holds the total
      const int first = cum - h.y;                                           // through this lane's first bin
      const bool in_first = first >= target;
      const int bstar = __shfl_sync(0xffffffffu, 2 * lane + (in_first ? 0 : 1), l0);
      c = __shfl_sync(0xffffffffu, in_first ? first : cum, l0);              // candidates in bins <= b*: the survivors
      keep = valid && bin <= bstar;
      const unsigned km = __ballot_sync(0xffffffffu, keep);
      local = __popc(km & ((1u << lane) - 1u));
      if (lane == 0) ss->wcount[warp] = __popc(km);
    }
    SEL_STAMP(4);
    asm volatile("bar.sync 1, %0;" ::"r"(n_active) : "memory");             // ---- barrier 2
    SEL_STAMP(5);
    // ---- step 3: pack the survivors, warp after warp
    {
      const int off = __reduce_add_sync(0xffffffffu, lane < warp ? ss->wcount[lane] : 0);
      if (keep) ss->surv[off + local] = key;
      if (tid == 0) ss->surv[c] = kPadKey;            // the rank loop reads the list in pairs; a pad precedes nothing
      if (tid < 64) ss->hist[tid] = 0;                // for the next call (this call's readers are past barrier 2)
    }
    SEL_STAMP(6);
    asm volatile("bar.sync 1, %0;" ::"r"(n_active) : "memory");             // ---- barrier 3
    SEL_STAMP(7);
    // ---- step 4: rank of a survivor = the survivors that precede it; 2^sh threads (adjacent lanes) share one count
    int sh = 0;
    while (sh < 3 && (c << (sh + 1)) <= n_active) ++sh;
    const int sv = tid >> sh, part = tid & ((1 << sh) - 1);
    const Key me = sv < c ? ss->surv[sv] : ~0ull;
    int r = 0;
    const ulonglong2* pairs = reinterpret_cast<const ulonglong2*>(ss->surv);
    const int npair = (c + 1) >> 1;
    for (int o = part; o < npair; o += 1 << sh) {     // (four loads in flight per thread were slower: the step is issue-bound)
      const ulonglong2 q = pairs[o];
      r += (q.x > me ? 1 : 0) + (q.y > me ? 1 : 0);
    }
    for (int o = 1; o < (1 << sh); o <<= 1) r += __shfl_xor_sync(0xffffffffu, r, o);
    if (sv < c && part == 0 && r < 64) emit(r, me, any);
    if (tid < 64 && tid >= c) emit(tid, kPadKey, any);   // fewer than 64 candidates in all: the rest are pads
#ifdef DART_TREE_TL
    if (threadIdx.x == 0) g_sel_tl[10] = c;
#endif
  }
  SEL_STAMP(8);
  during4();
  __syncthreads();                                                          // ---- barrier 4
  return any;
}

}  // namespace dart
