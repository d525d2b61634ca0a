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
//     so all of them are looked up in one parallel sweep before the level loop; inside the
//     loop each candidate needs one trigram probe, whose context only exists once the
//     previous level's beam is known;
//   * top-w and top-theta use ranks, not sorts.  Every warp sorts its 32 candidates with a
//     shuffle bitonic network (total order: score desc, generation index asc).  A threshold
//     entry T is then taken from the runs' p-th entries: T = the m-th best of them with
//     m * (p + 1) >= theta, so at least theta candidates are not after T.  Only those
//     "survivors" (each run contributes a prefix; typically ~90 of 500) are ranked, by
//     counting the survivors that precede each one.  Ranks are unique, so "rank r < w" *is*
//     beam slot r and "rank r < theta" is the level's r-th finalist, with no dependence on
//     thread timing;
//   * the final top-theta only needs each level's theta best nodes (by ancestor-clamped
//     score): at most levels * theta finalists, ranked by the same counting.
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

// Finish a lookup whose first slot has been loaded: follow the probe sequence (bounded).
__device__ __forceinline__ bool probe_rest(const NgramTable& T, unsigned long long key, uint32_t h, NgramSlot s, float& score) {
  for (uint32_t i = 0; i <= T.max_probe; ++i) {
    if (s.key == key) { score = s.score; return true; }
    if (s.key == 0ull) return false;
    s = load_slot(T.slots + ((h + i + 1) & T.mask));
  }
  return false;
}

// (score, index) total order: a strictly precedes b
__device__ __forceinline__ bool before(float sa, int ia, float sb, int ib) { return sa > sb || (sa == sb && ia < ib); }

// Sort one value per lane so that lane 0 holds the entry that precedes all others.
__device__ __forceinline__ void warp_sort(float& s, int& c, int lane) {
#pragma unroll
  for (int k = 2; k <= 32; k <<= 1) {
#pragma unroll
    for (int j = k >> 1; j > 0; j >>= 1) {
      const float os = __shfl_xor_sync(0xffffffffu, s, j);
      const int oc = __shfl_xor_sync(0xffffffffu, c, j);
      const bool up = (lane & k) == 0, lower = (lane & j) == 0;
      const bool mine_first = before(s, c, os, oc);
      const bool keep = (lower == up) ? mine_first : !mine_first;
      if (!keep) { s = os; c = oc; }
    }
  }
}

// number of entries of a sorted 32-entry run that precede (s, c)
__device__ __forceinline__ int count_before(const float* rs, const int* rc, float s, int c) {
  int cnt = 0;
#pragma unroll
  for (int step = 32; step > 0; step >>= 1)
    if (cnt + step <= 32 && before(rs[cnt + step - 1], rc[cnt + step - 1], s, c)) cnt += step;
  return cnt;
}

struct TreeSmem {
  float* n_score; float* n_clamp; int* n_tok; int* n_par; unsigned char* n_j;
  float* bg; float* run_s; int* run_c; float* sv_s; int* sv_c; int* beam_a; int* beam_b; int* fin; int* sel; int* par_out; int* lvl_base;
};

__host__ __device__ inline size_t tree_layout(int k, int w, int budget, int L, unsigned char* base, TreeSmem* t) {
  const int n_max = 1 + k + (L - 1) * w * k;
  const int theta = budget - 1;
  size_t o = 0;
  auto take = [&](size_t bytes) { const size_t r = o; o += (bytes + 15) & ~size_t(15); return r; };
  const size_t o_score = take((size_t)n_max * 4), o_clamp = take((size_t)n_max * 4), o_tok = take((size_t)n_max * 4),
               o_par = take((size_t)n_max * 4), o_j = take((size_t)n_max), o_bg = take((size_t)(k + (L - 1) * k * k) * 4),
               o_rs = take(32 * 32 * 4), o_rc = take(32 * 32 * 4), o_ss = take(1024 * 4), o_sc = take(1024 * 4), o_ba = take((size_t)w * 4), o_bb = take((size_t)w * 4),
               o_fin = take((size_t)L * theta * 4), o_sel = take((size_t)budget * 4), o_po = take((size_t)budget * 4),
               o_lb = take((size_t)(L + 1) * 4);
  if (t != nullptr) {
    t->n_score = reinterpret_cast<float*>(base + o_score); t->n_clamp = reinterpret_cast<float*>(base + o_clamp);
    t->n_tok = reinterpret_cast<int*>(base + o_tok); t->n_par = reinterpret_cast<int*>(base + o_par);
    t->n_j = base + o_j; t->bg = reinterpret_cast<float*>(base + o_bg);
    t->run_s = reinterpret_cast<float*>(base + o_rs); t->run_c = reinterpret_cast<int*>(base + o_rc);
    t->sv_s = reinterpret_cast<float*>(base + o_ss); t->sv_c = reinterpret_cast<int*>(base + o_sc);
    t->beam_a = reinterpret_cast<int*>(base + o_ba); t->beam_b = reinterpret_cast<int*>(base + o_bb);
    t->fin = reinterpret_cast<int*>(base + o_fin); t->sel = reinterpret_cast<int*>(base + o_sel);
    t->par_out = reinterpret_cast<int*>(base + o_po); t->lvl_base = reinterpret_cast<int*>(base + o_lb);
  }
  return o;
}

__global__ void __launch_bounds__(1024) tree_kernel(const TreeParams p) {
  extern __shared__ __align__(16) unsigned char tsm[];
  const int k = p.topk, w = p.beam, L = p.n_levels, theta = p.budget - 1;
  TreeSmem m;
  tree_layout(k, w, p.budget, L, tsm, &m);
  __shared__ int s_nsurv, s_thr_c;
  __shared__ float s_thr_s;
  __shared__ unsigned long long s_bits[64];

  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int* ids = p.ids + ((size_t)b * p.K + p.first_row) * k;
  const float* sl = p.slogit + ((size_t)b * p.K + p.first_row) * k;
  const int ctx0 = p.ctx_tail[2 * b], ctx1 = p.ctx_tail[2 * b + 1];
  const NgramTable T = p.table;
  const bool have_table = T.slots != nullptr;

  if (tid == 0) {
    m.n_score[0] = 0.f; m.n_clamp[0] = INFINITY; m.n_tok[0] = ctx1; m.n_par[0] = -1; m.n_j[0] = 0;
    m.beam_a[0] = 0; m.lvl_base[0] = 1;
  }
  // ---- every bigram any level can ask for: bg[0][0][jt] = (ctx1, S_0[jt]); bg[i][jb][jt] = (S_{i-1}[jb], S_i[jt])
  {
    const int n_bg = k + (L - 1) * k * k;
    for (int base = 0; base < n_bg; base += 8 * 1024) {
      unsigned long long key[8];
      uint32_t hh[8];
      NgramSlot first[8];
      bool want[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int e = base + u * 1024 + tid;
        want[u] = false;
        if (e < n_bg && have_table) {
          int tb, tt;
          if (e < k) { tb = ctx1; tt = ids[e]; }
          else { const int r = e - k, i = 1 + r / (k * k), q = r % (k * k); tb = ids[(i - 1) * k + q / k]; tt = ids[i * k + q % k]; }
          if (tb >= 0) {
            key[u] = ngram_key(2, -1, tb, tt);
            hh[u] = (uint32_t)ngram_hash(key[u]) & T.mask;
            first[u] = load_slot(T.slots + hh[u]);
            want[u] = true;
          }
        }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int e = base + u * 1024 + tid;
        if (e < n_bg) {
          float sc = p.miss;
          if (want[u]) { float v; if (probe_rest(T, key[u], hh[u], first[u], v)) sc = v; }
          m.bg[e] = sc;
        }
      }
    }
  }
  __syncthreads();

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
      float s_ng = m.bg[i == 0 ? j : k + (i - 1) * k * k + (int)m.n_j[node] * k + j];
      if (have_table && p.ngram_order >= 3 && ta >= 0 && tb >= 0) {
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
    // does any candidate's clamped score differ from its score?  (never, when increments are <= 0)
    const int differs = __syncthreads_or(tid < ncand && cl != s);

    // ---- ranks by (score desc, generation asc); a second pass on the clamped scores only if they differ
    const int n_want = theta > w ? theta : w;
    for (int pass = 0; pass < (differs ? 2 : 1); ++pass) {
      float key = (pass == 0) ? s : cl;
      int c = (tid < ncand) ? tid : 0x7fffffff;
      if (warp < nruns) {
        warp_sort(key, c, lane);
        m.run_s[warp * 32 + lane] = key;
        m.run_c[warp * 32 + lane] = c;
      }
      if (tid == 0) s_nsurv = 0;
      __syncthreads();
      // threshold: the m-th best of the runs' p-th entries, m * (p + 1) >= n_want
      // (with too few runs for that, T is the sentinel that nothing is after: everything survives)
      int mm = (nruns + 1) >> 1;
      if (mm < ((n_want + 31) >> 5)) mm = (n_want + 31) >> 5;
      const int pp = (n_want + mm - 1) / mm - 1;
      if (warp == 0) {
        float tk = (lane < nruns) ? m.run_s[lane * 32 + pp] : -INFINITY;
        int tc = (lane < nruns) ? m.run_c[lane * 32 + pp] : 0x7fffffff;
        warp_sort(tk, tc, lane);
        if (mm > nruns) { tk = -INFINITY; tc = 0x7fffffff; }
        if (lane == (mm > nruns ? 0 : mm - 1)) { s_thr_s = tk; s_thr_c = tc; }
      }
      __syncthreads();
      const float ts = s_thr_s;
      const int tc = s_thr_c;
      // survivors: entries that are not after T (a prefix of every run)
      const bool surv = warp < nruns && c != 0x7fffffff && !before(ts, tc, key, c);
      const unsigned bal = __ballot_sync(0xffffffffu, surv);
      int off = 0;
      if (lane == 0 && bal) off = atomicAdd(&s_nsurv, __popc(bal));
      off = __shfl_sync(0xffffffffu, off, 0);
      if (surv) {
        const int slot = off + __popc(bal & ((1u << lane) - 1));
        m.sv_s[slot] = key;
        m.sv_c[slot] = c;
      }
      __syncthreads();
      const int ns = s_nsurv;
      if (surv) {
        int rank = 0;
        for (int o = 0; o < ns; ++o) rank += before(m.sv_s[o], m.sv_c[o], key, c);
        if (pass == 0) {
          if (rank < w) beam_next[rank] = base + c;
          if (!differs && rank < theta) m.fin[i * theta + rank] = base + c;
        } else if (rank < theta) {
          m.fin[i * theta + rank] = base + c;
        }
      }
      __syncthreads();
    }
    if (tid == 0) m.lvl_base[i + 1] = base + ncand;
    __syncthreads();
    nb = ncand < w ? ncand : w;
    int* tmp = beam; beam = beam_next; beam_next = tmp;
  }

  // ---- global top-theta over the per-level finalists (clamped score desc, node index asc)
  const int total = m.lvl_base[L] - 1;
  const int n_sel = total < theta ? total : theta;
  {
    // compact the finalists: level i contributes min(ncand_i, theta) nodes
    const int i = tid / theta, q = tid - i * theta;
    bool mine = false;
    int me = 0;
    if (i < L) {
      const int ncand_i = m.lvl_base[i + 1] - m.lvl_base[i];
      if (q < (ncand_i < theta ? ncand_i : theta)) { mine = true; me = m.fin[tid]; }
    }
    if (tid == 0) s_nsurv = 0;
    __syncthreads();
    const unsigned bal = __ballot_sync(0xffffffffu, mine);
    int off = 0;
    if (lane == 0 && bal) off = atomicAdd(&s_nsurv, __popc(bal));
    off = __shfl_sync(0xffffffffu, off, 0);
    float mc = 0.f;
    if (mine) {
      const int slot = off + __popc(bal & ((1u << lane) - 1));
      mc = m.n_clamp[me];
      m.sv_s[slot] = mc;
      m.sv_c[slot] = me;
    }
    __syncthreads();
    const int ns = s_nsurv;
    if (mine) {
      int rank = 0;
      for (int o = 0; o < ns; ++o) rank += before(m.sv_s[o], m.sv_c[o], mc, me);
      if (rank < n_sel) m.sel[rank + 1] = me;
    }
  }
  if (tid == 0) m.sel[0] = 0;
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
  for (int e = tid; e < budget * budget; e += 1024) {
    const int x = e / budget, y = e - x * budget;
    mbase[e] = (uint8_t)((s_bits[x] >> y) & 1ull);
  }
}

size_t tree_smem_bytes(int topk, int beam, int budget, int n_levels) {
  return tree_layout(topk, beam, budget, n_levels, nullptr, nullptr) + 16;
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
