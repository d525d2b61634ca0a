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

struct TreeSmem {
  float* n_score; float* n_clamp; int* n_tok; int* n_par; unsigned char* n_j;
  float* bg; Key* xk; int* beam_a; int* beam_b; int* sel; int* par_out; int* lvl_base;
};

__host__ __device__ inline size_t tree_layout(int k, int w, int budget, int L, unsigned char* base, TreeSmem* t) {
  const int n_max = 1 + k + (L - 1) * w * k;
  size_t o = 0;
  auto take = [&](size_t bytes) { const size_t r = o; o += (bytes + 15) & ~size_t(15); return r; };
  const size_t o_score = take((size_t)n_max * 4), o_clamp = take((size_t)n_max * 4), o_tok = take((size_t)n_max * 4),
               o_par = take((size_t)n_max * 4), o_j = take((size_t)n_max), o_bg = take((size_t)(k + (L - 1) * k * k) * 4),
               o_xk = take(32 * 64 * 8), o_ba = take((size_t)w * 4), o_bb = take((size_t)w * 4),
               o_sel = take((size_t)(budget + 1) * 4), o_po = take((size_t)budget * 4), o_lb = take((size_t)(L + 1) * 4);
  if (t != nullptr) {
    t->n_score = reinterpret_cast<float*>(base + o_score); t->n_clamp = reinterpret_cast<float*>(base + o_clamp);
    t->n_tok = reinterpret_cast<int*>(base + o_tok); t->n_par = reinterpret_cast<int*>(base + o_par);
    t->n_j = base + o_j; t->bg = reinterpret_cast<float*>(base + o_bg);
    t->xk = reinterpret_cast<Key*>(base + o_xk);
    t->beam_a = reinterpret_cast<int*>(base + o_ba); t->beam_b = reinterpret_cast<int*>(base + o_bb);
    t->sel = reinterpret_cast<int*>(base + o_sel);
    t->par_out = reinterpret_cast<int*>(base + o_po); t->lvl_base = reinterpret_cast<int*>(base + o_lb);
  }
  return o;
}

// Best 64 of the block's candidates (one key per thread; pads are kPadKey), sorted, in warp 0's (x0, x1).
// `pred` is OR-reduced over the block in the first barrier and returned.  nruns = warps that hold
// candidates.  All threads of the block must call this.
__device__ __forceinline__ int block_best64(Key key, int nruns, const TreeSmem& m, int pred, Key& x0, Key& x1) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  warp_sort(key, lane);
  x0 = key;
  x1 = kPadKey;
  int any = 0;
  bool first = true;
  for (int stride = 1; stride < nruns || first; stride <<= 1) {
    const bool donor = (warp & (2 * stride - 1)) == stride && warp < nruns;
    if (donor) {
      m.xk[warp * 64 + lane] = x0;
      m.xk[warp * 64 + 32 + lane] = x1;
    }
    if (first) { any = __syncthreads_or(pred); first = false; } else __syncthreads();
    if ((warp & (2 * stride - 1)) == 0 && warp + stride < nruns) {
      const int pw = (warp + stride) * 64;
      x0 = kmax(x0, m.xk[pw + 63 - lane]);
      x1 = kmax(x1, m.xk[pw + 31 - lane]);
      bitonic_merge64(x0, x1, lane);
    }
  }
  return any;
}

// MAXT: launch bound (512 leaves the compiler twice the registers; 1024 covers beam * topk up to 1024)
template <int MAXT>
__global__ void __launch_bounds__(MAXT) tree_kernel(const TreeParams p) {
  extern __shared__ __align__(16) unsigned char tsm[];
  const int k = p.topk, w = p.beam, L = p.n_levels, theta = p.budget - 1;
  TreeSmem m;
  tree_layout(k, w, p.budget, L, tsm, &m);
  __shared__ unsigned long long s_bits[64];

  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthr = blockDim.x;
  pdl_wait();
  const int* ids = p.ids + ((size_t)b * p.K + p.first_row) * k;
  const float* sl = p.slogit + ((size_t)b * p.K + p.first_row) * k;
  const int ctx0 = p.ctx_tail[2 * b], ctx1 = p.ctx_tail[2 * b + 1];
  const NgramTable T = p.table;
  const bool have_table = T.slots != nullptr;

  if (tid == 0) {
    m.n_score[0] = 0.f; m.n_clamp[0] = INFINITY; m.n_tok[0] = ctx1; m.n_par[0] = -1; m.n_j[0] = 0;
    m.beam_a[0] = 0; m.lvl_base[0] = 1;
  }
  // ---- every bigram any level can ask for: bg[jt] = (ctx1, S_0[jt]); bg[k + (i-1)k^2 + jb*k + jt] = (S_{i-1}[jb], S_i[jt]).
  // A thread issues the first probe of all its lookups (up to 12) before it resolves any of them.
  {
    const int n_bg = k + (L - 1) * k * k;
    for (int e0 = 0; e0 < n_bg; e0 += 12 * nthr) {
      Key key[12];
      uint32_t hh[12];
      NgramSlot first[12];
#pragma unroll
      for (int u = 0; u < 12; ++u) {
        const int e = e0 + u * nthr + tid;
        int tb = -1, tt = 0;
        if (e < n_bg) {
          if (e < k) { tb = ctx1; tt = ids[e]; }
          else { const int r = e - k, i = r / (k * k), q = r - i * k * k, jb = q / k; tb = ids[i * k + jb]; tt = ids[(i + 1) * k + q - jb * k]; }
        }
        const bool want = have_table && tb >= 0;
        key[u] = want ? ngram_key(2, -1, tb, tt) : 0ull;
        hh[u] = (uint32_t)ngram_hash(key[u]) & T.mask;
        first[u] = want ? load_slot(T.slots + hh[u]) : NgramSlot{0ull, 0.f, 0u};
      }
#pragma unroll
      for (int u = 0; u < 12; ++u) {
        const int e = e0 + u * nthr + tid;
        if (e < n_bg) {
          float sc = p.miss, v;
          if (key[u] != 0ull && probe_rest(T, key[u], hh[u], first[u], v)) sc = v;
          m.bg[e] = sc;
        }
      }
    }
  }
  __syncthreads();

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
    // keys carry the node index base + tid, which orders candidates of one level like tid does
    // best 64 by score -> next beam; `differs`: some clamped score is not its score (never, when increments <= 0)
    Key x0, x1;
    const int differs = block_best64(tid < ncand ? make_key(s, base + tid) : kPadKey, nruns, m, tid < ncand && cl != s, x0, x1);
    if (warp == 0 && lane < w && x0 != kPadKey) beam_next[lane] = key_index(x0);
    if (differs) {  // the level's best 64 by clamped score are a different set: select again
      __syncthreads();
      block_best64(tid < ncand ? make_key(cl, base + tid) : kPadKey, nruns, m, 0, x0, x1);
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

size_t tree_smem_bytes(int topk, int beam, int budget, int n_levels) {
  return tree_layout(topk, beam, budget, n_levels, nullptr, nullptr) + 16;
}

cudaError_t tree_setup(int topk, int beam, int budget, int max_levels) {
  const size_t smem = tree_smem_bytes(topk, beam, budget, max_levels);
  if (smem > 48 * 1024)
  {
    cudaError_t e = cudaFuncSetAttribute(tree_kernel<512>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(tree_kernel<1024>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  }
  return cudaSuccess;
}

cudaError_t launch_tree(const TreeParams& p, cudaStream_t st) {
  const size_t smem = tree_smem_bytes(p.topk, p.beam, p.budget, p.n_levels);
  // one thread per (beam entry, candidate) pair; a smaller block makes every barrier cheaper
  int need = p.beam * p.topk;
  if (p.budget > need) need = p.budget;
  int threads = (need + 31) / 32 * 32;
  if (threads > 1024) threads = 1024;
  if (threads <= 512) return launch_pdl(tree_kernel<512>, dim3(p.B), dim3(threads), smem, st, p);
  return launch_pdl(tree_kernel<1024>, dim3(p.B), dim3(threads), smem, st, p);
}

}  // namespace dart
