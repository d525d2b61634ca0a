// Continuity-aware tree pruning (Algorithm 1, Appendix D) -- one thread block per sequence.
//
// Per level, one thread per (beam entry, candidate) pair scores the extension:
//   s' = sc + ((w_logit * s_logit) + (w_ng * s_ng)) * w_level
// with s_ng read from an open-addressing hash table of N-gram rows (trigram, then bigram,
// then log(eps)).  All score arithmetic is fp32 round-to-nearest with no fused multiply-add
// (__fmul_rn/__fadd_rn), in the same order as a sequential evaluation, so the tree is
// bit-exact with one.
//
// Latency is what matters here (a few thousand candidates, a few hundred random 16-byte reads):
//   * every bigram a level can ask for is known up front -- (token of S_{i-1}, token of S_i) --
//     so all of them are looked up by a separate many-block kernel first (one SM cannot keep
//     4400 random reads in flight; 13 us inside this kernel against ~2 us spread over the GPU);
//     inside the level loop each candidate needs one trigram probe, whose context only exists
//     once the previous level's beam is known;
//   * selection is a bitonic merge tree held in registers.  Every warp sorts its 32 candidates
//     with a shuffle network (total order: score desc, generation index asc); pairs of warps
//     then merge their runs, keeping the best 64 (two per lane): C[p] = better(A[p], B[63-p])
//     is a bitonic sequence holding the best 64 of A and B, which six compare-exchange stages
//     sort.  After log2(warps) rounds warp 0 holds the level's best 64 in order: the first w
//     are the next beam (w <= 32).  There are no data-dependent loops and the result does
//     not depend on thread timing;
//   * the final top-theta (theta <= 63) is kept the same way: warp 0 merges each level's best
//     64 (by ancestor-clamped score, node index asc) into a running global best 64.
#include "common.cuh"
#include "kernels.h"
#include "select.cuh"

namespace dart {

__device__ __forceinline__ NgramSlot load_slot(const NgramSlot* p) {
  const uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
  NgramSlot s;
  s.key = ((unsigned long long)v.y << 32) | v.x;
  s.score = __uint_as_float(v.z);
  s.pad = v.w;
  return s;
}

// Finish a lookup whose first slot has been loaded: follow the probe sequence (bounded).
__device__ __forceinline__ bool probe_rest(const NgramTable& T, unsigned long long key, uint32_t h, NgramSlot s, float& score) {
  for (uint32_t i = 0; i <= T.max_probe; ++i) {
    if (s.key == key) { score = s.score; return true; }
    if (s.key == 0ull) return false;
    s = load_slot(T.slots + ((h + i + 1) & T.mask));
  }
  return false;
}

// Look `key` up in the sorted list ent[lo .. hi) of {key, payload} pairs (a child list of the trie, at most 2^21
// entries).  A 16-ary search: every round reads 15 evenly spaced keys at once -- their latencies overlap, so a round
// costs one memory round trip -- and keeps the sixteenth of the list that can hold the key; a list of 16 or fewer is
// read whole.  1 round trip for the common short list, 5 for a list as long as the vocabulary.  The rounds are
// bounded and every read stays inside [lo, hi), whatever the list holds.
__device__ __forceinline__ bool trie_find(const uint2* __restrict__ ent, uint32_t lo, uint32_t hi, int key, uint32_t& payload, uint32_t& index) {
#pragma unroll 1
  for (int round = 0; round < 6 && hi - lo > 16u; ++round) {
    const uint32_t n = hi - lo;
    int piv[15];
#pragma unroll
    for (int q = 0; q < 15; ++q) piv[q] = (int)__ldg(&ent[lo + ((n * (uint32_t)(q + 1)) >> 4)].x);
    uint32_t c = 0;
#pragma unroll
    for (int q = 0; q < 15; ++q) c += piv[q] <= key ? 1u : 0u;
    const uint32_t nlo = lo + ((n * c) >> 4), nhi = c < 15u ? lo + ((n * (c + 1u)) >> 4) : hi;
    lo = nlo; hi = nhi;
  }
  bool found = false;
#pragma unroll
  for (int q = 0; q < 16; ++q) {
    const uint32_t idx = lo + (uint32_t)q;
    if (idx < hi) {
      const uint2 v = __ldg(&ent[idx]);
      if ((int)v.x == key) { found = true; payload = v.y; index = idx; }
    }
  }
  return found;
}

// Sizes of the per-sequence sweep outputs: bigram scores and 3-gram context ranges for `levels` levels.
__host__ __device__ inline int sweep_bigrams(int k, int levels) { return k + (levels - 1) * k * k; }
__host__ __device__ inline int sweep_contexts(int k, int levels) { return 1 + (levels >= 2 ? k : 0) + (levels > 2 ? (levels - 2) * k * k : 0); }

struct TreeSmem {
  float* n_score; float* n_clamp; int* n_tok; int* n_par; unsigned char* n_j;
  Key* xk; int* beam_a; int* beam_b; int* sel; int* par_out; int* lvl_base;
};

__host__ __device__ inline size_t tree_layout(int k, int w, int budget, int L, unsigned char* base, TreeSmem* t) {
  const int n_max = 1 + k + (L - 1) * w * k;
  size_t o = 0;
  auto take = [&](size_t bytes) { const size_t r = o; o += (bytes + 15) & ~size_t(15); return r; };
  const size_t o_score = take((size_t)n_max * 4), o_clamp = take((size_t)n_max * 4), o_tok = take((size_t)n_max * 4),
               o_par = take((size_t)n_max * 4), o_j = take((size_t)n_max),
               o_xk = take(32 * 64 * 8), o_ba = take((size_t)w * 4), o_bb = take((size_t)w * 4),
               o_sel = take((size_t)(budget + 1) * 4), o_po = take((size_t)budget * 4), o_lb = take((size_t)(L + 1) * 4);
  if (t != nullptr) {
    t->n_score = reinterpret_cast<float*>(base + o_score); t->n_clamp = reinterpret_cast<float*>(base + o_clamp);
    t->n_tok = reinterpret_cast<int*>(base + o_tok); t->n_par = reinterpret_cast<int*>(base + o_par);
    t->n_j = base + o_j;
    t->xk = reinterpret_cast<Key*>(base + o_xk);
    t->beam_a = reinterpret_cast<int*>(base + o_ba); t->beam_b = reinterpret_cast<int*>(base + o_bb);
    t->sel = reinterpret_cast<int*>(base + o_sel);
    t->par_out = reinterpret_cast<int*>(base + o_po); t->lvl_base = reinterpret_cast<int*>(base + o_lb);
  }
  return o;
}

// Bigram scores of every (level, previous candidate, candidate) triple, one lookup per thread:
// bg[b][jt] = (ctx1, S_0[jt]) for e < k, bg[b][k + (i-1)k^2 + jb*k + jt] = (S_{i-1}[jb], S_i[jt]); a missing row
// gives log(eps).
__global__ void __launch_bounds__(256) bigram_sweep_kernel(const TreeParams p) {
  pdl_wait();
  const int k = p.topk, b = blockIdx.y;
  const int fr = p.first_rows[b], Lb = min(p.n_levels, p.K - fr);   // this sequence's level 0 row and levels
  const int n_bg = k + (p.n_levels - 1) * k * k;                   // layout stride: the launch's maximum
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= k + (Lb - 1) * k * k) return;
  const int* ids = p.ids + ((size_t)b * p.K + fr) * k;
  int tb, tt;
  if (e < k) { tb = p.ctx_tail[2 * b + 1]; tt = ids[e]; }
  else { const int r = e - k, i = r / (k * k), q = r - i * k * k, jb = q / k; tb = ids[i * k + jb]; tt = ids[(i + 1) * k + q - jb * k]; }
  float sc = p.miss;
  if (p.table.slots != nullptr && tb >= 0) {
    const unsigned long long key = ngram_key(2, -1, tb, tt);
    const uint32_t hh = (uint32_t)ngram_hash(key) & p.table.mask;
    float v;
    if (probe_rest(p.table, key, hh, load_slot(p.table.slots + hh), v)) sc = v;
  }
  p.bg[(size_t)b * n_bg + e] = sc;
}

// The sweep for the trie layout.  Besides the bigram scores (a search of context b's child list for t) it locates
// the node of every 3-gram context a level can ask for -- (c_-2, c_-1) for level 0, (c_-1, S_0[j]) for level 1,
// (S_{i-2}[j'], S_{i-1}[j]) for level i -- once, and leaves the range of its children in cx, laid out like bg:
// cx[b][0], cx[b][1 + j], cx[b][1 + k + (i-2)k^2 + j'k + j].  A context that is absent gets the empty range.
__global__ void __launch_bounds__(256) trie_sweep_kernel(const TreeParams p) {
  pdl_wait();
  const int k = p.topk, b = blockIdx.y;
  const int fr = p.first_rows[b], Lb = min(p.n_levels, p.K - fr);
  const int n_bg = sweep_bigrams(k, p.n_levels), n_cx = sweep_contexts(k, p.n_levels);   // layout strides: the launch's maximum
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  const int* ids = p.ids + ((size_t)b * p.K + fr) * k;
  const NgramTrie T = p.trie;
  uint32_t pay, idx;
  if (e < n_bg) {
    if (e >= sweep_bigrams(k, Lb)) return;
    int tb, tt;
    if (e < k) { tb = p.ctx_tail[2 * b + 1]; tt = ids[e]; }
    else { const int r = e - k, i = r / (k * k), q = r - i * k * k, jb = q / k; tb = ids[i * k + jb]; tt = ids[(i + 1) * k + q - jb * k]; }
    float sc = p.miss;
    if (tb >= 0 && tb < p.vocab && trie_find(T.bi_ent, __ldg(T.bi_off + tb), __ldg(T.bi_off + tb + 1), tt, pay, idx)) sc = __uint_as_float(pay);
    p.bg[(size_t)b * n_bg + e] = sc;
    return;
  }
  const int c = e - n_bg;
  if (c >= sweep_contexts(k, Lb)) return;
  int ta, tb;
  if (c == 0) { ta = p.ctx_tail[2 * b]; tb = p.ctx_tail[2 * b + 1]; }
  else if (c < 1 + k) { ta = p.ctx_tail[2 * b + 1]; tb = ids[c - 1]; }
  else { const int r = c - 1 - k, i2 = r / (k * k), q = r - i2 * k * k, jp = q / k; ta = ids[i2 * k + jp]; tb = ids[(i2 + 1) * k + q - jp * k]; }
  uint2 range = make_uint2(0u, 0u);
  if (p.ngram_order >= 3 && ta >= 0 && ta < p.vocab && tb >= 0 && trie_find(T.tri_node, __ldg(T.tri_off + ta), __ldg(T.tri_off + ta + 1), tb, pay, idx))
    range = make_uint2(pay, __ldg(&T.tri_node[idx + 1]).y);
  p.cx[(size_t)b * n_cx + c] = range;
}

// MAXT: launch bound (512 leaves the compiler twice the registers; 1024 covers beam * topk up to 1024)
// TRIE: the N-gram is the child-list trie (3-gram scores: search the context's children, located by the sweep).
template <int MAXT, bool TRIE>
__global__ void __launch_bounds__(MAXT) tree_kernel(const TreeParams p) {
  extern __shared__ __align__(16) unsigned char tsm[];
  const int k = p.topk, w = p.beam, theta = p.budget - 1;
  const int fr = p.first_rows[blockIdx.x], L = min(p.n_levels, p.K - fr);   // this sequence's level 0 row and levels
  TreeSmem m;
  tree_layout(k, w, p.budget, p.n_levels, tsm, &m);
  __shared__ unsigned long long s_bits[64];

  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthr = blockDim.x;
  pdl_wait();
  const int* ids = p.ids + ((size_t)b * p.K + fr) * k;
  const float* sl = p.slogit + ((size_t)b * p.K + fr) * k;
  const int ctx0 = p.ctx_tail[2 * b], ctx1 = p.ctx_tail[2 * b + 1];
  const NgramTable T = p.table;
  const bool have_table = T.slots != nullptr;
  const float* bg = p.bg + (size_t)b * sweep_bigrams(k, p.n_levels);  // bigram scores from the sweep kernel
  const uint2* cx = TRIE ? p.cx + (size_t)b * sweep_contexts(k, p.n_levels) : nullptr;

  if (tid == 0) {
    m.n_score[0] = 0.f; m.n_clamp[0] = INFINITY; m.n_tok[0] = ctx1; m.n_par[0] = -1; m.n_j[0] = 0;
    m.beam_a[0] = 0; m.lvl_base[0] = 1;
  }
  // running global best 64 by (clamped score desc, node index asc); lives in warp 0's registers
  Key g0 = kPadKey, g1 = kPadKey;

  int nb = 1;
  int* beam = m.beam_a;
  int* beam_next = m.beam_b;
  for (int i = 0; i < L; ++i) {
    const int ncand = nb * k;
    const int base = m.lvl_base[i];
    const int nruns = (ncand + 31) >> 5;
    float s = -INFINITY, cl = -INFINITY;
    if (tid < ncand) {
      const int rho = tid / k, j = tid - rho * k;
      const int node = beam[rho];
      const int tb = m.n_tok[node];
      const int ta = node == 0 ? ctx0 : m.n_tok[m.n_par[node]];
      const int t = ids[i * k + j];
      float s_ng = __ldg(bg + (i == 0 ? j : k + (i - 1) * k * k + (int)m.n_j[node] * k + j));
      if (TRIE) {
        const int jn = m.n_j[node];
        const int c = i == 0 ? 0 : i == 1 ? 1 + jn : 1 + k + (i - 2) * k * k + (int)m.n_j[m.n_par[node]] * k + jn;
        const uint2 range = __ldg(cx + c);
        uint32_t pay, idx;
        if (range.y > range.x && trie_find(p.trie.tri_ent, range.x, range.y, t, pay, idx)) s_ng = __uint_as_float(pay);
      } else if (have_table && p.ngram_order >= 3 && ta >= 0 && tb >= 0) {
        const unsigned long long k3 = ngram_key(3, ta, tb, t);
        const uint32_t h3 = (uint32_t)ngram_hash(k3) & T.mask;
        float v;
        if (probe_rest(T, k3, h3, load_slot(T.slots + h3), v)) s_ng = v;
      }
      const float inc = __fmul_rn(__fadd_rn(__fmul_rn(p.wl[i], sl[i * k + j]), __fmul_rn(p.wn, s_ng)), p.wv[i]);
      s = __fadd_rn(m.n_score[node], inc);
      const float pc = m.n_clamp[node];
      cl = s < pc ? s : pc;
      const int n = base + tid;
      m.n_score[n] = s; m.n_clamp[n] = cl; m.n_tok[n] = t; m.n_par[n] = node; m.n_j[n] = (unsigned char)j;
    }
    // keys carry the node index base + tid, which orders candidates of one level like tid does
    // best 64 by score -> next beam; `differs`: some clamped score is not its score (never, when increments <= 0)
    Key x0, x1;
    const int differs = block_best64(tid < ncand ? make_key(s, base + tid) : kPadKey, nruns, m.xk, tid < ncand && cl != s, x0, x1);
    if (warp == 0 && lane < w && x0 != kPadKey) beam_next[lane] = key_index(x0);
    if (differs) {  // the level's best 64 by clamped score are a different set: select again
      __syncthreads();
      block_best64(tid < ncand ? make_key(cl, base + tid) : kPadKey, nruns, m.xk, 0, x0, x1);
    }
    if (warp == 0) merge_keep64(g0, g1, x0, x1, lane);
    if (tid == 0) m.lvl_base[i + 1] = base + ncand;
    __syncthreads();
    nb = ncand < w ? ncand : w;
    int* tmp = beam; beam = beam_next; beam_next = tmp;
  }

  // ---- the selected nodes: the first n_sel entries of the global best 64
  const int total = m.lvl_base[L] - 1;
  const int n_sel = total < theta ? total : theta;
  if (warp == 0) {
    if (lane < n_sel) m.sel[1 + lane] = key_index(g0);
    if (32 + lane < n_sel) m.sel[33 + lane] = key_index(g1);
    if (lane == 0) m.sel[0] = 0;
  }
  __syncthreads();

  // ---- outputs
  const int budget = p.budget;
  if (tid < budget) {
    int po = -1;
    if (tid >= 1 && tid <= n_sel) {
      const int pn = m.n_par[m.sel[tid]];
      po = 0;
      if (pn != 0)
        for (int x = 1; x <= n_sel; ++x)
          if (m.sel[x] == pn) { po = x; break; }
    }
    m.par_out[tid] = po;
  }
  __syncthreads();
  if (tid < budget) {
    const size_t o = (size_t)b * budget + tid;
    unsigned long long bits = 0ull;
    if (tid <= n_sel) {
      const int n = m.sel[tid];
      int lev = 0;
      if (tid > 0) {
        while (n >= m.lvl_base[lev + 1]) ++lev;
        lev += 1;
      }
      p.tokens[o] = m.n_tok[n];
      p.parents[o] = m.par_out[tid];
      p.depth[o] = lev;
      if (p.scores) p.scores[o] = tid == 0 ? 0.f : m.n_clamp[n];
      int x = tid;
      for (int guard = 0; guard <= L + 1 && x >= 0; ++guard) { bits |= 1ull << x; x = m.par_out[x]; }
    } else {
      p.tokens[o] = -1; p.parents[o] = -1; p.depth[o] = -1;
      if (p.scores) p.scores[o] = -INFINITY;
    }
    s_bits[tid] = bits;
  }
  if (tid == 0) p.n_nodes[b] = 1 + n_sel;
  __syncthreads();
  uint8_t* mbase = p.mask + (size_t)b * budget * budget;
  for (int e = tid; e < budget * budget; e += nthr) {
    const int x = e / budget, y = e - x * budget;
    mbase[e] = (uint8_t)((s_bits[x] >> y) & 1ull);
  }
}

// Verification inputs of one tree per block: thread x owns slot x (budget <= 64 threads' worth of slots).
__global__ void __launch_bounds__(64) verify_inputs_kernel(int budget, int max_levels, const int32_t* parents, const int32_t* depth,
                                                           const int32_t* n_nodes, const int32_t* root_pos, int32_t* position_ids,
                                                           int32_t* retrieve, int32_t* n_leaves) {
  __shared__ int s_par[64], s_dep[64], s_isp[64];
  const int b = blockIdx.x, x = threadIdx.x, W = max_levels + 1;
  pdl_wait();
  const int n = n_nodes[b];
  const bool used = x < n && x < budget;
  s_par[x] = used ? parents[(size_t)b * budget + x] : -1;
  s_dep[x] = used ? depth[(size_t)b * budget + x] : -1;
  s_isp[x] = 0;
  __syncthreads();
  if (used && x >= 1 && s_par[x] >= 0 && s_par[x] < 64) s_isp[s_par[x]] = 1;   // benign race: every writer stores 1
  __syncthreads();
  if (x < budget) position_ids[(size_t)b * budget + x] = used ? root_pos[b] + s_dep[x] : -1;
  const bool leaf = used && !s_isp[x];
  int rank = 0, total = 0;
  for (int y = 0; y < budget && y < 64; ++y) {
    const int l = (y < n && !s_isp[y]) ? 1 : 0;
    total += l;
    if (y < x) rank += l;
  }
  int32_t* rows = retrieve + (size_t)b * budget * W;
  if (x < budget && x >= total)   // rows past the last leaf are all -1: row x is cleared by thread x
    for (int c = 0; c < W; ++c) rows[(size_t)x * W + c] = -1;
  if (leaf) {
    int32_t* row = rows + (size_t)rank * W;
    const int d = s_dep[x];
    for (int c = d + 1; c < W; ++c) row[c] = -1;
    int y = x;
    for (int guard = 0; guard <= max_levels && y >= 0; ++guard) {   // bounded walk up the parent chain
      const int dy = s_dep[y];
      if (dy >= 0 && dy < W) row[dy] = y;
      y = s_par[y];
    }
  }
  if (x == 0) n_leaves[b] = total;
}

cudaError_t launch_verify_inputs(int B, int budget, int max_levels, const int32_t* parents, const int32_t* depth, const int32_t* n_nodes,
                                 const int32_t* root_pos, int32_t* position_ids, int32_t* retrieve, int32_t* n_leaves, cudaStream_t st) {
  return launch_pdl(verify_inputs_kernel, dim3(B), dim3(64), 0, st, budget, max_levels, parents, depth, n_nodes, root_pos, position_ids,
                    retrieve, n_leaves);
}

size_t tree_smem_bytes(int topk, int beam, int budget, int n_levels) {
  return tree_layout(topk, beam, budget, n_levels, nullptr, nullptr) + 16;
}

cudaError_t tree_setup(int topk, int beam, int budget, int max_levels) {
  const size_t smem = tree_smem_bytes(topk, beam, budget, max_levels);
  if (smem > 48 * 1024)
  {
    cudaError_t e = cudaFuncSetAttribute(tree_kernel<512, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(tree_kernel<1024, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(tree_kernel<512, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(tree_kernel<1024, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    return e;
  }
  return cudaSuccess;
}

cudaError_t launch_tree(const TreeParams& p, cudaStream_t st) {
  const bool trie = p.trie.bi_off != nullptr;
  {
    const int n_bg = sweep_bigrams(p.topk, p.n_levels), n_cx = sweep_contexts(p.topk, p.n_levels);
    cudaError_t e = trie ? launch_pdl(trie_sweep_kernel, dim3((n_bg + n_cx + 255) / 256, p.B), dim3(256), 0, st, p)
                         : launch_pdl(bigram_sweep_kernel, dim3((n_bg + 255) / 256, p.B), dim3(256), 0, st, p);
    if (e != cudaSuccess) return e;
  }
  const size_t smem = tree_smem_bytes(p.topk, p.beam, p.budget, p.n_levels);
  // one thread per (beam entry, candidate) pair; a smaller block makes every barrier cheaper
  int need = p.beam * p.topk;
  if (p.budget > need) need = p.budget;
  int threads = (need + 31) / 32 * 32;
  if (threads > 1024) threads = 1024;
  if (trie) {
    if (threads <= 512) return launch_pdl(tree_kernel<512, true>, dim3(p.B), dim3(threads), smem, st, p);
    return launch_pdl(tree_kernel<1024, true>, dim3(p.B), dim3(threads), smem, st, p);
  }
  if (threads <= 512) return launch_pdl(tree_kernel<512, false>, dim3(p.B), dim3(threads), smem, st, p);
  return launch_pdl(tree_kernel<1024, false>, dim3(p.B), dim3(threads), smem, st, p);
}

}  // namespace dart
