// Merge of the LM head's per-CTA results into the final candidates of one logit row
// (Algorithm 1 lines 6-8: S_i = top-k tokens, s_logit = log(softmax + eps), Appendix D).
//
// Input per CTA c and token row: (max, sum-exp) of its vocab slice and its best `topk` entries
// (selection key, plain logit y, token id), sorted by (key desc, id asc).  One block per token row:
//   1. log-sum-exp over the slices (fixed-order reductions, deterministic);
//   2. all G lists (keys, ids, plain logits) are copied to shared memory with coalesced loads, all requested at once;
//   3. a threshold T taken from the list *heads*: the heads are warp-sorted and T = the m-th best of
//      the runs' p-th entries with m * (p + 1) >= topk, so at least topk heads are not after T and the
//      global top-k lies among the entries that are not after T; each sorted list contributes a prefix;
//   4. every survivor (typically a few dozen) counts the survivors that precede it: its rank, and, below topk,
//      its place in the output.
// Nothing here depends on the order in which threads run.
#include "common.cuh"
#include "kernels.h"
#include "select.cuh"

namespace dart {

constexpr int kMergeThreads = 512;
constexpr int kMergeYsMaxGrid = 256;   // up to this many lists their plain logits fit in shared memory beside the rest

__global__ void __launch_bounds__(kMergeThreads) topk_merge_kernel(const LmParams p) {
  extern __shared__ __align__(16) unsigned char msm[];
  const int G = p.grid, MP = padded_tokens(p.M), tk = blockIdx.x, topk = p.topk;
  float* keys = reinterpret_cast<float*>(msm);                 // [G*32]
  int* ids = reinterpret_cast<int*>(keys + G * 32);            // [G*32]
  const bool has_ys = G <= kMergeYsMaxGrid;
  float* ys = reinterpret_cast<float*>(ids + G * 32);          // [G*32] plain logits (if they fit)
  Key* skey = reinterpret_cast<Key*>(ys + (has_ys ? G * 32 : 0));   // [G*32] survivors' keys
  int* ssrc = reinterpret_cast<int*>(skey + G * 32);           // [G*32] survivors' positions c*32+e
  Key* xk = reinterpret_cast<Key*>(ssrc + G * 32);             // [16 warps][64] merge-tree scratch
  Key* hr = xk + 16 * 64;                                      // [32 runs][32] sorted heads
  __shared__ float sh_m[16], sh_s[16];
  __shared__ float s_lse;
  __shared__ Key s_thr;
  __shared__ int s_nsurv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_wait();
  pdl_trigger();   // a short kernel: the next one may be scheduled and run its set-up now

  // Every global load of the kernel is requested before any is used (the lists' keys, ids and plain logits with
  // coalesced 16-byte loads, the slices' statistics), so the kernel pays one round trip to memory, not one per loop
  // iteration or per phase.
  float m = -INFINITY, s = 0.f;
  {
    const float4* ksrc = reinterpret_cast<const float4*>(p.part_key);
    const float4* ysrc = reinterpret_cast<const float4*>(p.part_y);
    const int4* isrc = reinterpret_cast<const int4*>(p.part_id);
    constexpr int kBatch = 3;
    for (int base = 0; base < G * 8; base += kBatch * kMergeThreads) {
      float4 kr[kBatch], yr[kBatch];
      int4 ir[kBatch];
#pragma unroll
      for (int q = 0; q < kBatch; ++q) {
        const int i = base + q * kMergeThreads + tid;
        if (i < G * 8) {
          const size_t o = ((size_t)(i >> 3) * MP + tk) * 8 + (i & 7);
          kr[q] = ksrc[o];
          if (has_ys) yr[q] = ysrc[o];
          ir[q] = isrc[o];
        }
      }
      float mc = -INFINITY, sc = 0.f;
      // ---- log-sum-exp over the slices: per-thread online (max, sum), combined in a fixed order below
      const int c0 = base / 8 + tid;   // the slices whose lists this pass copies: base/8 .. base/8 + kBatch*64 - 1
      const bool has = tid < kBatch * (kMergeThreads / 8) && c0 < G;
      if (has) { mc = p.part_stats[((size_t)c0 * MP + tk) * 2]; sc = p.part_stats[((size_t)c0 * MP + tk) * 2 + 1]; }
#pragma unroll
      for (int q = 0; q < kBatch; ++q) {
        const int i = base + q * kMergeThreads + tid;
        if (i < G * 8) {
          reinterpret_cast<float4*>(keys)[i] = kr[q];
          if (has_ys) reinterpret_cast<float4*>(ys)[i] = yr[q];
          reinterpret_cast<int4*>(ids)[i] = ir[q];
        }
      }
      if (has && mc != -INFINITY) {
        const float mn = fmaxf(m, mc);
        s = s * expf(m - mn) + sc * expf(mc - mn);
        m = mn;
      }
    }
  }
  if (tid == 0) s_nsurv = 0;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float mo = __shfl_xor_sync(0xffffffffu, m, o), so = __shfl_xor_sync(0xffffffffu, s, o);
    const float mn = fmaxf(m, mo);
    const float a = (m == -INFINITY) ? 0.f : s * expf(m - mn), b = (mo == -INFINITY) ? 0.f : so * expf(mo - mn);
    // both lanes of a pair compute the same value (addition is commutative)
    s = a + b;
    m = mn;
  }
  if (lane == 0) { sh_m[warp] = m; sh_s[warp] = s; }
  __syncthreads();   // also publishes keys/ids
  if (tid == 0) {
    float mm = -INFINITY;
    for (int i = 0; i < kMergeThreads / 32; ++i) mm = fmaxf(mm, sh_m[i]);
    float ss = 0.f;
    for (int i = 0; i < kMergeThreads / 32; ++i)
      if (sh_m[i] != -INFINITY) ss += sh_s[i] * expf(sh_m[i] - mm);
    s_lse = mm + logf(ss);
  }

  // ---- threshold from the list heads
  const int nruns = (G + 31) >> 5;  // <= 32
  Key hk = kPadKey;
  if (tid < nruns * 32) {
    const int c = tid;
    if (c < G && keys[c * 32] != -INFINITY) hk = make_key(keys[c * 32], ids[c * 32]);
    warp_sort(hk, lane);
    hr[warp * 32 + lane] = hk;
  }
  __syncthreads();
  if (warp == 0) {
    int mm = (nruns + 1) >> 1;
    const int pp = (topk + mm - 1) / mm - 1;   // <= 31 because topk <= 32
    Key t = (lane < nruns) ? hr[lane * 32 + pp] : kPadKey;
    warp_sort(t, lane);
    t = shfl_key(t, mm - 1);
    if (lane == 0) s_thr = t;
  }
  __syncthreads();
  const Key thr = s_thr;

  // ---- survivors: the prefix of every sorted list that is not after the threshold
  for (int c = tid; c < G; c += kMergeThreads) {
    for (int e = 0; e < topk; ++e) {
      const float k = keys[c * 32 + e];
      if (k == -INFINITY) break;
      const Key kk = make_key(k, ids[c * 32 + e]);
      if (kk < thr) break;
      const int slot = atomicAdd(&s_nsurv, 1);
      skey[slot] = kk;
      ssrc[slot] = c * 32 + e;
    }
  }
  __syncthreads();
  const int ns = s_nsurv;
  const float lse = s_lse;
  const int filled = ns < topk ? ns : topk;

  {
    // ---- rank every survivor by counting the survivors that precede it (typically a few dozen of them: the count is
    // a short loop of broadcast reads on two or three warps; a sort network over the block cost several times that)
    for (int sidx = tid; sidx < ns; sidx += kMergeThreads) {
      const Key me = skey[sidx];
      int rank = 0;
#pragma unroll 4
      for (int o = 0; o < ns; ++o) rank += skey[o] > me ? 1 : 0;
      if (rank < topk) {
        const int src = ssrc[sidx];
        const float y = has_ys ? ys[src] : p.part_y[((size_t)(src >> 5) * MP + tk) * 32 + (src & 31)];
        p.out_ids[(size_t)tk * topk + rank] = ids[src];
        p.out_slogit[(size_t)tk * topk + rank] = logf(expf(y - lse) + p.eps_logit);
      }
    }
  }
  if (tid >= filled && tid < topk) {
    p.out_ids[(size_t)tk * topk + tid] = -1;
    p.out_slogit[(size_t)tk * topk + tid] = -INFINITY;
  }
}

static size_t merge_smem(int G) { return (size_t)G * 32 * (4 + 4 + (G <= kMergeYsMaxGrid ? 4 : 0) + 8 + 4) + (16 * 64 + 32 * 32) * 8 + 64; }

cudaError_t topk_merge_setup(int max_grid) {
  size_t smem = merge_smem(max_grid);
  if (max_grid > kMergeYsMaxGrid && merge_smem(kMergeYsMaxGrid) > smem) smem = merge_smem(kMergeYsMaxGrid);
  if (smem > 48 * 1024)
    return cudaFuncSetAttribute(topk_merge_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  return cudaSuccess;
}

cudaError_t launch_topk_merge(const LmParams& p, cudaStream_t st) {
  return launch_pdl(topk_merge_kernel, dim3(p.M), dim3(kMergeThreads), merge_smem(p.grid), st, p);
}

}  // namespace dart
