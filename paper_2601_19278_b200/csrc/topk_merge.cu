// Merge of the LM head's per-CTA results into the final candidates of one logit row
// (Algorithm 1 lines 6-8: S_i = top-k tokens, s_logit = log(softmax + eps), Appendix D).
//
// Input per CTA c and token row: (max, sum-exp) of its vocab slice and its best `topk` entries
// (selection key, plain logit y, token id), sorted by (key desc, id asc).  One block per token row:
//   1. log-sum-exp over the slices (fixed-order reductions, deterministic);
//   2. all G lists are copied to shared memory with coalesced loads;
//   3. a threshold T = the topk-th best of the G list *heads* (at least topk entries are >= T, so
//      the global top-k lies among the entries >= T; each sorted list contributes a prefix);
//   4. the survivors (typically a few dozen) are ranked by counting how many survivors precede
//      each one in the total order (key desc, id asc); rank r < topk is output slot r.
// Nothing here depends on the order in which threads run.
#include "common.cuh"
#include "kernels.h"

namespace dart {

__device__ __forceinline__ bool cand_before(float ka, int ia, float kb, int ib) {  // a strictly precedes b
  return ka > kb || (ka == kb && ia < ib);
}

__global__ void __launch_bounds__(1024) topk_merge_kernel(const LmParams p) {
  extern __shared__ __align__(16) unsigned char msm[];
  const int G = p.grid, MP = padded_tokens(p.M), tk = blockIdx.x, topk = p.topk;
  float* keys = reinterpret_cast<float*>(msm);        // [G*32]
  int* ids = reinterpret_cast<int*>(keys + G * 32);   // [G*32]
  int* surv = ids + G * 32;                           // [G*32]
  __shared__ float sh[32];
  __shared__ float s_thr_key;
  __shared__ int s_thr_id, s_nsurv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthr = blockDim.x;
  pdl_wait();

  for (int i = tid; i < G * 32; i += nthr) {
    const int c = i >> 5, e = i & 31;
    const size_t o = ((size_t)c * MP + tk) * 32 + e;
    keys[i] = (e < topk) ? p.part_key[o] : -INFINITY;
    ids[i] = p.part_id[o];
  }
  if (tid == 0) { s_thr_key = -INFINITY; s_thr_id = 0x7fffffff; s_nsurv = 0; }

  // ---- log-sum-exp over the slices
  float mx = -INFINITY;
  for (int c = tid; c < G; c += nthr) mx = fmaxf(mx, p.part_stats[((size_t)c * MP + tk) * 2]);
  mx = warp_max(mx);
  __syncthreads();
  if (lane == 0) sh[warp] = mx;
  __syncthreads();
  mx = sh[0];
  for (int i = 1; i < (nthr >> 5); ++i) mx = fmaxf(mx, sh[i]);
  float sum = 0.f;
  for (int c = tid; c < G; c += nthr) {
    const float mc = p.part_stats[((size_t)c * MP + tk) * 2];
    if (mc != -INFINITY) sum += p.part_stats[((size_t)c * MP + tk) * 2 + 1] * expf(mc - mx);
  }
  sum = block_sum(sum, sh);
  const float lse = mx + logf(sum);

  // ---- threshold from the list heads
  if (G >= topk) {
    for (int c = tid; c < G; c += nthr) {
      const float mk = keys[c * 32];
      const int mi = ids[c * 32];
      int rank = 0;
      for (int o = 0; o < G; ++o) rank += cand_before(keys[o * 32], ids[o * 32], mk, mi);
      if (rank == topk - 1) { s_thr_key = mk; s_thr_id = mi; }
    }
  }
  __syncthreads();
  const float tkey = s_thr_key;
  const int tidx = s_thr_id;

  // ---- survivors: the prefix of every sorted list that is not after the threshold entry
  for (int c = tid; c < G; c += nthr) {
    for (int e = 0; e < topk; ++e) {
      const float k = keys[c * 32 + e];
      if (k == -INFINITY || cand_before(tkey, tidx, k, ids[c * 32 + e])) break;
      surv[atomicAdd(&s_nsurv, 1)] = c * 32 + e;
    }
  }
  __syncthreads();
  const int ns = s_nsurv;

  // ---- rank the survivors; rank r < topk is output slot r
  for (int s = tid; s < ns; s += nthr) {
    const int me = surv[s];
    const float mk = keys[me];
    const int mi = ids[me];
    int rank = 0;
    for (int o = 0; o < ns; ++o) {
      const int ot = surv[o];
      rank += cand_before(keys[ot], ids[ot], mk, mi);
    }
    if (rank < topk) {
      const int c = me >> 5, e = me & 31;
      const float y = p.part_y[((size_t)c * MP + tk) * 32 + e];
      p.out_ids[(size_t)tk * topk + rank] = mi;
      p.out_slogit[(size_t)tk * topk + rank] = logf(expf(y - lse) + p.eps_logit);
    }
  }
  const int filled = ns < topk ? ns : topk;
  if (tid >= filled && tid < topk) {
    p.out_ids[(size_t)tk * topk + tid] = -1;
    p.out_slogit[(size_t)tk * topk + tid] = -INFINITY;
  }
}

static size_t merge_smem(int G) { return (size_t)G * 32 * 12; }

cudaError_t topk_merge_setup(int max_grid) {
  const size_t smem = merge_smem(max_grid);
  if (smem > 48 * 1024)
    return cudaFuncSetAttribute(topk_merge_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  return cudaSuccess;
}

cudaError_t launch_topk_merge(const LmParams& p, cudaStream_t st) {
  return launch_pdl(topk_merge_kernel, dim3(p.M), dim3(1024), merge_smem(p.grid), st, p);
}

}  // namespace dart
