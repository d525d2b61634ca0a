// Continuity-aware tree pruning (Algorithm 1, Appendix D) -- one thread block per sequence.
//
// Per level, one thread per (beam entry, candidate) pair scores the extension:
//   s' = sc + ((w_logit * s_logit) + (w_ng * s_ng)) * w_level
// with s_ng read from an open-addressing hash table of N-gram rows (trigram, then bigram,
// then log(eps)).  All score arithmetic is fp32 round-to-nearest with no fused multiply-add
// (__fmul_rn/__fadd_rn), in the same order as a sequential evaluation, so the tree is
// bit-exact with one.  Top-w and the final top-theta are taken by *rank counting*: a
// candidate's rank is the number of candidates that precede it in the total order
// (score desc, generation index asc), which is deterministic and needs no sort.  For the
// final selection only each level's theta best nodes (by ancestor-clamped score) can matter,
// so the global ranking runs over at most levels * theta nodes.
#include "common.cuh"
#include "kernels.h"

namespace dart {

__device__ __forceinline__ NgramSlot load_slot(const NgramSlot* p) {
  const uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
  NgramSlot s;
  s.key = ((unsigned long long)v.y << 32) | v.x;
  s.score = __uint_as_float(v.z);
  s.pad = v.w;
  return s;
}

// s_ng for context (a, b) and token t: trigram row, else bigram row, else `miss`.
__device__ float ngram_score_dev(const NgramTable& T, int order, int a, int b, int t, float miss) {
  if (T.slots == nullptr || b < 0) return miss;
  const bool try3 = order >= 3 && a >= 0;
  const unsigned long long k3 = ngram_key(3, a, b, t), k2 = ngram_key(2, -1, b, t);
  const uint32_t h3 = (uint32_t)ngram_hash(k3) & T.mask, h2 = (uint32_t)ngram_hash(k2) & T.mask;
  // both first probes are independent loads
  NgramSlot s3 = load_slot(T.slots + (try3 ? h3 : h2));
  NgramSlot s2 = load_slot(T.slots + h2);
  if (try3) {
    for (uint32_t i = 0; i <= T.max_probe; ++i) {
      if (s3.key == k3) return s3.score;
      if (s3.key == 0ull) break;
      s3 = load_slot(T.slots + ((h3 + i + 1) & T.mask));
    }
  }
  for (uint32_t i = 0; i <= T.max_probe; ++i) {
    if (s2.key == k2) return s2.score;
    if (s2.key == 0ull) break;
    s2 = load_slot(T.slots + ((h2 + i + 1) & T.mask));
  }
  return miss;
}

__global__ void __launch_bounds__(1024) tree_kernel(const TreeParams p) {
  extern __shared__ __align__(16) unsigned char tsm[];
  const int k = p.topk, w = p.beam, L = p.n_levels, theta = p.budget - 1;
  const int n_max = 1 + k + (L - 1) * w * k;
  const int cmax = w * k > k ? w * k : k;
  float* n_score = reinterpret_cast<float*>(tsm);            // [n_max]
  float* n_clamp = n_score + n_max;                            // [n_max]
  int* n_tok = reinterpret_cast<int*>(n_clamp + n_max);        // [n_max]
  int* n_par = n_tok + n_max;                                  // [n_max]
  float* c_s = reinterpret_cast<float*>(n_par + n_max);        // [cmax] level scratch: scores
  float* c_cl = c_s + cmax;                                    // [cmax] clamped scores
  int* beam_a = reinterpret_cast<int*>(c_cl + cmax);           // [w]
  int* beam_b = beam_a + w;                                    // [w]
  int* fin = beam_b + w;                                       // [L*theta] final-selection candidates (node ids)
  int* sel = fin + L * theta;                                  // [budget] selected node per output slot
  int* par_out = sel + p.budget;                               // [budget]
  int* lvl_base = par_out + p.budget;                          // [L+1]

  const int b = blockIdx.x, tid = threadIdx.x;
  const int* ids = p.ids + ((size_t)b * p.K + p.first_row) * k;
  const float* sl = p.slogit + ((size_t)b * p.K + p.first_row) * k;
  const int ctx0 = p.ctx_tail[2 * b], ctx1 = p.ctx_tail[2 * b + 1];

  if (tid == 0) {
    n_score[0] = 0.f; n_clamp[0] = INFINITY; n_tok[0] = ctx1; n_par[0] = -1;
    beam_a[0] = 0; lvl_base[0] = 1;
  }
  __syncthreads();

  int nb = 1;
  int* beam = beam_a;
  int* beam_next = beam_b;
  for (int i = 0; i < L; ++i) {
    const int ncand = nb * k;
    const int base = lvl_base[i];
    float s = 0.f, cl = 0.f;
    if (tid < ncand) {
      const int rho = tid / k, j = tid - rho * k;
      const int node = beam[rho];
      const int tb = n_tok[node];
      const int ta = node == 0 ? ctx0 : n_tok[n_par[node]];
      const int t = ids[i * k + j];
      const float s_logit = sl[i * k + j];
      const float s_ng = ngram_score_dev(p.table, p.ngram_order, ta, tb, t, p.miss);
      const float inc = __fmul_rn(__fadd_rn(__fmul_rn(p.wl[i], s_logit), __fmul_rn(p.wn, s_ng)), p.wv[i]);
      s = __fadd_rn(n_score[node], inc);
      const float pc = n_clamp[node];
      cl = s < pc ? s : pc;
      const int n = base + tid;
      n_score[n] = s; n_clamp[n] = cl; n_tok[n] = t; n_par[n] = node;
      c_s[tid] = s; c_cl[tid] = cl;
    }
    __syncthreads();
    if (tid < ncand) {
      int rank_beam = 0, rank_fin = 0;
      for (int c = 0; c < ncand; ++c) {
        const float os = c_s[c], oc = c_cl[c];
        rank_beam += (os > s) || (os == s && c < tid);
        rank_fin += (oc > cl) || (oc == cl && c < tid);
      }
      if (rank_beam < w) beam_next[rank_beam] = base + tid;
      if (rank_fin < theta) fin[i * theta + rank_fin] = base + tid;
    }
    if (tid == 0) {
      lvl_base[i + 1] = base + ncand;
    }
    __syncthreads();
    nb = ncand < w ? ncand : w;
    int* tmp = beam; beam = beam_next; beam_next = tmp;
  }

  // ---- global top-theta over the per-level finalists (clamped score desc, node index asc)
  // finalists of level i occupy fin[i*theta .. i*theta + min(ncand_i, theta))
  int my_node = -1;
  {
    const int i = tid / theta, rk = tid - i * theta;
    if (i < L) {
      const int ncand_i = lvl_base[i + 1] - lvl_base[i];
      if (rk < (ncand_i < theta ? ncand_i : theta)) my_node = fin[tid];
    }
  }
  int total = lvl_base[L] - 1;
  const int n_sel = total < theta ? total : theta;
  if (my_node >= 0) {
    const float cl = n_clamp[my_node];
    int rank = 0;
    for (int i = 0; i < L; ++i) {
      const int ncand_i = lvl_base[i + 1] - lvl_base[i];
      const int cnt = ncand_i < theta ? ncand_i : theta;
      for (int q = 0; q < cnt; ++q) {
        const int o = fin[i * theta + q];
        const float oc = n_clamp[o];
        rank += (oc > cl) || (oc == cl && o < my_node);
      }
    }
    if (rank < n_sel) sel[rank + 1] = my_node;
  }
  if (tid == 0) sel[0] = 0;
  __syncthreads();

  // ---- outputs
  const int budget = p.budget;
  if (tid < budget) {
    int po = -1;
    if (tid >= 1 && tid <= n_sel) {
      const int pn = n_par[sel[tid]];
      po = 0;
      if (pn != 0)
        for (int x = 1; x <= n_sel; ++x)
          if (sel[x] == pn) { po = x; break; }
    }
    par_out[tid] = po;
  }
  __syncthreads();
  if (tid < budget) {
    const size_t o = (size_t)b * budget + tid;
    if (tid <= n_sel) {
      const int n = sel[tid];
      int lev = 0;
      if (tid > 0) {
        while (n >= lvl_base[lev + 1]) ++lev;
        lev += 1;
      }
      p.tokens[o] = n_tok[n];
      p.parents[o] = par_out[tid];
      p.depth[o] = lev;
      if (p.scores) p.scores[o] = tid == 0 ? 0.f : n_clamp[n];
      unsigned long long bits = 0ull;
      int x = tid;
      for (int guard = 0; guard <= L + 1 && x >= 0; ++guard) { bits |= 1ull << x; x = par_out[x]; }
      uint8_t* mrow = p.mask + o * budget;
      for (int y = 0; y < budget; ++y) mrow[y] = (uint8_t)((bits >> y) & 1ull);
    } else {
      p.tokens[o] = -1; p.parents[o] = -1; p.depth[o] = -1;
      if (p.scores) p.scores[o] = -INFINITY;
      uint8_t* mrow = p.mask + o * budget;
      for (int y = 0; y < budget; ++y) mrow[y] = 0;
    }
  }
  if (tid == 0) p.n_nodes[b] = 1 + n_sel;
}

size_t tree_smem_bytes(int topk, int beam, int budget, int n_levels) {
  const int n_max = 1 + topk + (n_levels - 1) * beam * topk;
  const int cmax = beam * topk > topk ? beam * topk : topk;
  const int theta = budget - 1;
  return (size_t)n_max * 16 + (size_t)cmax * 8 + (size_t)beam * 8 + (size_t)n_levels * theta * 4 + (size_t)budget * 8 +
         (size_t)(n_levels + 1) * 4 + 64;
}

cudaError_t tree_setup(int topk, int beam, int budget, int max_levels) {
  const size_t smem = tree_smem_bytes(topk, beam, budget, max_levels);
  if (smem > 48 * 1024)
    return cudaFuncSetAttribute(tree_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  return cudaSuccess;
}

cudaError_t launch_tree(const TreeParams& p, cudaStream_t st) {
  const size_t smem = tree_smem_bytes(p.topk, p.beam, p.budget, p.n_levels);
  tree_kernel<<<p.B, 1024, smem, st>>>(p);
  return cudaGetLastError();
}

}  // namespace dart
