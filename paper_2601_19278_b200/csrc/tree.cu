// Continuity-aware tree pruning (Algorithm 1, Appendix D) -- one thread block per sequence.
//
// Per level, one thread per (beam entry, candidate) pair scores the extension:
//   s' = sc + ((w_logit * s_logit) + (w_ng * s_ng)) * w_level
// with s_ng read from an open-addressing hash table of N-gram rows (trigram, then bigram,
// then log(eps)).  All score arithmetic is fp32 round-to-nearest with no fused multiply-add
// (__fmul_rn/__fadd_rn), in the same order as a sequential evaluation, so the tree is
// bit-exact with one.
//
// Latency is what matters here (a few thousand candidates, a few hundred random 16-byte reads per level if they
// were made inside the level loop).  With the hash layout (ngram_sweep_kernel + tree_hash_kernel):
//   * every N-gram score a level can ask for is known before the first level runs -- the context of a level-i
//     candidate is (a token of S_{i-2}, a token of S_{i-1}) -- so a many-block sweep looks all of them up first
//     (k + k^2 + (levels-2) k^3 lookups: 94 400 at k = 25 and 8 levels, a few hundred per SM, one round trip) and
//     leaves the final s_ng (3-gram row, else 2-gram row, else log eps) in a dense table; the tree kernel copies
//     one level's slice of it (k^3 floats) into shared memory while the previous level is being selected, so the
//     level loop itself touches no global memory;
//   * the per-level selection is block_select64 of select.cuh (histogram threshold + rank counting, four barriers);
//   * the final top-theta (theta <= 63) is a running best 64 (by ancestor-clamped score, node index asc) that the
//     block's last warp merges one level behind, while the other warps rank the next level's survivors.
// With the trie layout (trie_sweep_kernel + tree_kernel) the 3-gram scores are read inside the level loop -- one warp
// per beam entry walks its context's child list -- and the selection is the register merge tree of select.cuh.
// Nothing depends on the order in which threads run.
#include "common.cuh"
#include "kernels.h"
#include "select.cuh"

namespace dart {

// The entry of token t in a long list (region ent[lo ..), nb8 bitmap slots first): read t's 64-byte bitmap block,
// test its bit, count the entries before it, read the entry -- two dependent reads whatever the list's length.
__device__ __forceinline__ bool long_find(const uint2* __restrict__ ent, uint32_t lo, uint32_t nb8, int t, uint32_t& payload, uint32_t& index) {
  const uint32_t blk = (uint32_t)t / 480u, r = (uint32_t)t - blk * 480u;
  if (blk * 8u >= nb8) return false;                       // a token beyond the vocabulary
  const uint4* bp = reinterpret_cast<const uint4*>(ent + lo + blk * 8u);
  const uint4 q0 = __ldg(bp), q1 = __ldg(bp + 1), q2 = __ldg(bp + 2), q3 = __ldg(bp + 3);
  const uint32_t w[16] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w, q2.x, q2.y, q2.z, q2.w, q3.x, q3.y, q3.z, q3.w};
  const uint32_t word = 1u + (r >> 5), bit = r & 31u;
  uint32_t rank = w[0], mine = 0u;
#pragma unroll
  for (uint32_t q = 1; q < 16; ++q) {
    rank += q < word ? (uint32_t)__popc(w[q]) : 0u;
    mine = q == word ? w[q] : mine;
  }
  if (((mine >> bit) & 1u) == 0u) return false;
  rank += (uint32_t)__popc(mine & ((1u << bit) - 1u));
  index = lo + nb8 + rank;
  payload = __ldg(&ent[index]).y;
  return true;
}

// The candidate tokens S_i of one level as a 64-slot open-addressing table in shared memory (k <= 32, so it is at
// most half full): token -> the first position j that holds it.  Built and read by one warp or, with a barrier
// between the two, by a block.
// `filter` is a 2048-bit map of the tokens' low bits: nearly every child of a list is not a candidate, and one
// read of the map says so.
struct CandSet { int tok[64]; int j[64]; uint32_t filter[64]; };

__device__ __forceinline__ uint32_t cand_slot(int t) { return ((uint32_t)t * 0x9E3779B1u) >> 26; }
__device__ __forceinline__ void cand_clear(CandSet& s, int lane) {
  s.tok[lane] = -1; s.tok[lane + 32] = -1; s.j[lane] = 0x7fffffff; s.j[lane + 32] = 0x7fffffff;
  s.filter[lane] = 0u; s.filter[lane + 32] = 0u;
}
__device__ __forceinline__ bool cand_maybe(const CandSet& s, int t) { return (s.filter[((uint32_t)t >> 5) & 63u] >> ((uint32_t)t & 31u)) & 1u; }
__device__ __forceinline__ void cand_insert(CandSet& s, int t, int j) {   // t >= 0
  atomicOr(&s.filter[((uint32_t)t >> 5) & 63u], 1u << ((uint32_t)t & 31u));
  uint32_t h = cand_slot(t);
  for (int probe = 0; probe < 64; ++probe, h = (h + 1) & 63u) {
    const int old = atomicCAS(&s.tok[h], -1, t);
    if (old == -1 || old == t) { atomicMin(&s.j[h], j); return; }
  }
}
__device__ __forceinline__ int cand_find(const CandSet& s, int t) {       // first j with token t, or -1
  uint32_t h = cand_slot(t);
  for (int probe = 0; probe < 64; ++probe, h = (h + 1) & 63u) {
    const int v = s.tok[h];
    if (v == t) return s.j[h];
    if (v == -1) return -1;
  }
  return -1;
}

// One warp intersects the child list in region ent[lo .. hi) with a candidate set (Appendix C: the context's node is
// reached once, its children are then read for all candidates).  A short list is read whole, 32 consecutive slots
// per instruction and sixteen instructions in flight together -- as many requests as the list has cache lines,
// one memory round trip per 512 slots, two at most -- and every child is looked up in the set.  In a long list
// each candidate's entry is found through the list's bitmap instead: lane j looks for my_t (its candidate's token
// where j is the token's first position, else -1).
// emit(j, payload, index) is called once per candidate token found, with j its first position.
// DEPTH: reads in flight per lane.
template <int DEPTH, typename Match, typename Emit>
__device__ __forceinline__ void warp_list_match(const uint2* __restrict__ ent, uint32_t lo, uint32_t hi, uint32_t nb8, Match match, int my_t,
                                                int lane, Emit emit) {
  if (hi <= lo) return;
  if (hi - lo <= (uint32_t)kTrieLongList + 7u) {
#pragma unroll 1
    for (uint32_t base = lo; base < hi; base += 32u * DEPTH) {
      uint2 v[DEPTH];
#pragma unroll
      for (int u = 0; u < DEPTH; ++u) {
        const uint32_t idx = base + (uint32_t)(u * 32 + lane);
        v[u] = idx < hi ? __ldg(&ent[idx]) : make_uint2(0xffffffffu, 0u);
      }
#pragma unroll
      for (int u = 0; u < DEPTH; ++u) {
        const int j = (int)v[u].x >= 0 ? match((int)v[u].x) : -1;
        if (j >= 0) emit(j, v[u].y, base + (uint32_t)(u * 32 + lane));
      }
    }
  } else if (my_t >= 0) {
    uint32_t pay, idx;
    if (long_find(ent, lo, nb8, my_t, pay, idx)) emit(lane, pay, idx);
  }
}

// Sizes of the per-sequence sweep outputs: bigram scores and 3-gram context ranges for `levels` levels.
__host__ __device__ inline int sweep_bigrams(int k, int levels) { return k + (levels - 1) * k * k; }
__host__ __device__ inline int sweep_contexts(int k, int levels) { return 1 + (levels >= 2 ? k : 0) + (levels > 2 ? (levels - 2) * k * k : 0); }

struct TreeSmem {
  float* n_score; float* n_clamp; int* n_tok; int* n_par; unsigned char* n_j;
  Key* xk; int* beam_a; int* beam_b; int* sel; int* par_out; int* lvl_base;
  // trie layout: per level the candidate set and every candidate's first position; per (beam entry, candidate)
  // the 3-gram score bits and per beam entry the mask of candidates that have one, double-buffered by level
  CandSet* sets; unsigned char* fj; uint32_t* s3; uint32_t* hit;
  uint2* cxs;   // [2][k*k] child ranges of the contexts the next level can ask for, copied in one level ahead
};

__host__ __device__ inline size_t tree_layout(int k, int w, int budget, int L, unsigned char* base, TreeSmem* t) {
  const int n_max = 1 + k + (L - 1) * w * k;
  size_t o = 0;
  auto take = [&](size_t bytes) { const size_t r = o; o += (bytes + 15) & ~size_t(15); return r; };
  const size_t o_score = take((size_t)n_max * 4), o_clamp = take((size_t)n_max * 4), o_tok = take((size_t)n_max * 4),
               o_par = take((size_t)n_max * 4), o_j = take((size_t)n_max),
               o_xk = take(32 * 64 * 8), o_ba = take((size_t)w * 4), o_bb = take((size_t)w * 4),
               o_sel = take((size_t)(budget + 1) * 4), o_po = take((size_t)budget * 4), o_lb = take((size_t)(L + 1) * 4),
               o_sets = take((size_t)L * sizeof(CandSet)), o_fj = take((size_t)L * k), o_s3 = take((size_t)2 * w * k * 4),
               o_hit = take(2 * 32 * 4), o_cxs = take((size_t)2 * k * k * 8);
  if (t != nullptr) {
    t->sets = reinterpret_cast<CandSet*>(base + o_sets); t->fj = base + o_fj;
    t->s3 = reinterpret_cast<uint32_t*>(base + o_s3); t->hit = reinterpret_cast<uint32_t*>(base + o_hit);
    t->cxs = reinterpret_cast<uint2*>(base + o_cxs);
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

// ---- dense N-gram score tables of one sequence (hash layout), written by the sweep ----
//   bg0  [j]                           2-gram (c_-1, S_0[j])
//   t0   [j]                           3-gram (c_-2, c_-1, S_0[j])
//   bg   [(i-1) k^2 + j' k + j]        2-gram (S_{i-1}[j'], S_i[j]), levels i >= 1
//   t1   [j' k + j]                    3-gram (c_-1, S_0[j'], S_1[j])
//   t3   [(i-2) st3 + (j'' k + j') k + j]   3-gram (S_{i-2}[j''], S_{i-1}[j'], S_i[j]), levels i >= 2: one slice per level
// A 2-gram entry holds the row's score or log(eps); a 3-gram entry the row's score or kNoRow, in which case the
// candidate's s_ng is its 2-gram entry (Algorithm 1 line 9 with Appendix C's back-off).  Offsets and strides are
// multiples of four floats so that tables can be copied with 16-byte cp.async; everything before t3 ("the small
// tables", 20 KB at k = 25 and 8 levels) is staged in shared memory once, t3 one slice at a time.
constexpr uint32_t kNoRowBits = 0x7fc00000u;   // a NaN: no score is one
struct SgLayout { int t0, bg, t1, small, st3, total; };
__host__ __device__ inline SgLayout sg_layout(int k, int levels) {
  SgLayout g;
  g.t0 = (k + 3) & ~3;
  g.bg = (g.t0 + k + 3) & ~3;
  g.t1 = (g.bg + (levels > 1 ? levels - 1 : 0) * k * k + 3) & ~3;
  g.small = (g.t1 + k * k + 3) & ~3;
  g.st3 = (k * k * k + 3) & ~3;
  g.total = g.small + (levels > 2 ? levels - 2 : 0) * g.st3;
  return g;
}
size_t tree_sg_floats(int topk, int levels) { return (size_t)sg_layout(topk, levels).total; }

// One lookup (see NgramTable): the fingerprint word of the key's home bucket; a slot is read (and its key compared)
// only where a fingerprint matches; a word with an empty slot and no matching row ends the search (a miss), a full one
// sends it on to the next bucket, at most max_probe times.
__device__ __noinline__ bool table_find(const NgramTable T, unsigned long long key, float* score) {
  const unsigned long long hh = ngram_hash(key);
  const uint32_t f = ngram_fingerprint(hh);
  uint32_t h = (uint32_t)hh & T.mask;
  for (uint32_t i = 0; i <= T.max_probe; ++i, h = (h + 1) & T.mask) {
    const uint4 w = __ldg(T.fp + h);
    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
    bool has_empty = false;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const uint32_t g = (ww[q >> 1] >> ((q & 1) * 16)) & 0xffffu;
      has_empty = has_empty || g == 0u;
      if (g == f) {
        const uint4 sl = __ldg(reinterpret_cast<const uint4*>(T.slots + (size_t)h * 8 + q));
        if ((((unsigned long long)sl.y << 32) | sl.x) == key) { *score = __uint_as_float(sl.z); return true; }
      }
    }
    if (has_empty) return false;
  }
  return false;
}

// The sweep's unit of work is one row of k entries, a warp per row and a lane per candidate of the level, so that the
// row's context tokens, its place in the tables and the level are worked out once per warp (one thread per entry spent
// most of its time on the divisions that take an entry's index apart: the sweep is bound by instructions, not by its
// reads -- the same 7.7 us with a table fresh in L2 as with a cold one).
//   small rows  r = 0: bg0 and t0;  r = 1 + (i-1) k + j', i >= 1: bg of (level i, j'), and for i = 1 also t1 of j'
//   slice rows  (level i >= 2, r' = j'' k + j'): t3
__host__ __device__ inline int sweep_small_rows(int k, int levels) { return 1 + (levels > 1 ? levels - 1 : 0) * k; }

__device__ __forceinline__ void sweep_lookup2(const TreeParams& p, int ta, int tb, int tt, float* dst2, float* dst3) {
  // dst2 (may be null): the 2-gram entry (tb, tt); dst3 (may be null): the 3-gram entry (ta, tb, tt)
  const bool have = p.table.slots != nullptr && tb >= 0;
  float v;
  if (dst2 != nullptr) *dst2 = (have && table_find(p.table, ngram_key(2, -1, tb, tt), &v)) ? v : p.miss;
  if (dst3 != nullptr)
    *dst3 = (have && p.ngram_order >= 3 && ta >= 0 && table_find(p.table, ngram_key(3, ta, tb, tt), &v))
                ? v : __uint_as_float(kNoRowBits);
}
__device__ __forceinline__ void sweep_small_row(const TreeParams& p, int b, int Lb, const SgLayout& g, int r, int lane) {
  const int k = p.topk;
  if (lane >= k) return;
  const int* ids = p.ids + ((size_t)b * p.K + p.first_rows[b]) * k;
  float* sg = p.sg + (size_t)b * g.total;
  if (r == 0) {
    sweep_lookup2(p, p.ctx_tail[2 * b], p.ctx_tail[2 * b + 1], ids[lane], sg + lane, sg + g.t0 + lane);
  } else {
    const int i = 1 + (r - 1) / k, j1 = (r - 1) - (i - 1) * k;
    if (i >= Lb) return;
    sweep_lookup2(p, i == 1 ? p.ctx_tail[2 * b + 1] : -1, ids[(i - 1) * k + j1], ids[i * k + lane], sg + g.bg + (i - 1) * k * k + j1 * k + lane,
                  i == 1 ? sg + g.t1 + j1 * k + lane : nullptr);
  }
}
__device__ __forceinline__ void sweep_slice_row(const TreeParams& p, int b, int Lb, const SgLayout& g, int i, int r, int lane) {
  const int k = p.topk;
  if (lane >= k || i >= Lb) return;
  const int* ids = p.ids + ((size_t)b * p.K + p.first_rows[b]) * k;
  const int j2 = r / k, j1 = r - j2 * k;
  sweep_lookup2(p, ids[(i - 2) * k + j2], ids[(i - 1) * k + j1], ids[i * k + lane], nullptr,
                p.sg + (size_t)b * g.total + g.small + (i - 2) * g.st3 + r * k + lane);
}

// The sweep as a kernel of its own (batches whose fused launch would not fit the GPU): one warp per row.
__global__ void __launch_bounds__(256) ngram_sweep_kernel(const TreeParams p) {
  pdl_wait();
  pdl_trigger();   // a short kernel: the next one may be scheduled and run its set-up now
  const int b = blockIdx.y, k = p.topk, lane = threadIdx.x & 31;
  const int Lb = min(p.n_levels, p.K - p.first_rows[b]);   // this sequence's levels
  const SgLayout g = sg_layout(k, p.n_levels);
  const int n_small = sweep_small_rows(k, p.n_levels), row = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row < n_small) sweep_small_row(p, b, Lb, g, row, lane);
  else {
    const int rr = row - n_small, i = 2 + rr / (k * k);
    if (i < p.n_levels) sweep_slice_row(p, b, Lb, g, i, rr - (i - 2) * k * k, lane);
  }
}

// The sweep for the trie layout: one warp per (level i, list kind, context position jb).  The context token x is
// c_-1 for level 0 and S_{i-1}[jb] after it; the warp intersects one of x's two child lists with S_i:
//   kind 0  the 2-gram children of x        -> bg, the bigram scores (x, S_i[j]);
//   kind 1  the 3-gram context nodes (x, .) -> cx, the child ranges of the contexts (x, S_i[j]) that level i+1 can
//           ask for, laid out like bg: cx[b][0] = (c_-2, c_-1), cx[b][1 + j] = (c_-1, S_0[j]),
//           cx[b][1 + k + (i-1)k^2 + jb k + j] = (S_{i-1}[jb], S_i[j]).  An absent context gets the empty range.
__global__ void __launch_bounds__(256) trie_sweep_kernel(const TreeParams p) {
  __shared__ CandSet s_set[8];
  pdl_wait();
  const int k = p.topk, b = blockIdx.y, lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const int fr = p.first_rows[b], Lb = min(p.n_levels, p.K - fr);
  const int task = blockIdx.x * 8 + wib;                 // ((i * 2) + kind) * k + jb
  const int i = task / (2 * k), kind = (task - i * 2 * k) / k, jb = task - (i * 2 + kind) * k;
  if (i >= Lb || (i == 0 && jb > 0)) return;
  const int* ids = p.ids + ((size_t)b * p.K + fr) * k;
  const NgramTrie T = p.trie;
  float* bg = p.bg + (size_t)b * sweep_bigrams(k, p.n_levels);
  uint2* cx = p.cx + (size_t)b * sweep_contexts(k, p.n_levels);
  const bool tri = p.ngram_order >= 3;
  if (kind == 1 && i == 0) {                             // the context of level 0
    const int ta = p.ctx_tail[2 * b], tb = p.ctx_tail[2 * b + 1];
    if (lane == 0) cx[0] = make_uint2(0u, 0u);
    __syncwarp();
    if (tri && ta >= 0 && ta < p.vocab && tb >= 0)
      warp_list_match<16>(T.tri_node, __ldg(T.tri_off + ta), __ldg(T.tri_off + ta + 1), T.nb8, [&](int tok) { return tok == tb ? 0 : -1; },
                      lane == 0 ? tb : -1, lane, [&](int, uint32_t pay, uint32_t idx) {
                        const uint2 range = make_uint2(pay, __ldg(&T.tri_node[idx + 1]).y);
                        cx[0] = range;
                      });
  }
  if (kind == 1 && i + 1 >= Lb) return;                  // no level left to ask for these contexts
  const int x = i == 0 ? p.ctx_tail[2 * b + 1] : ids[(i - 1) * k + jb];
  const int t = lane < k ? ids[i * k + lane] : -1;
  CandSet& set = s_set[wib];
  cand_clear(set, lane);
  __syncwarp();
  if (t >= 0) cand_insert(set, t, lane);
  __syncwarp();
  const int fj = t >= 0 ? cand_find(set, t) : lane;      // first position of this lane's token
  const bool have = x >= 0 && x < p.vocab && (kind == 0 || tri);
  if (kind == 0) {
    float* out = bg + (i == 0 ? 0 : k + (i - 1) * k * k + jb * k);
    if (lane < k) out[lane] = p.miss;
    __syncwarp();
    if (have)
      warp_list_match<16>(T.bi_ent, __ldg(T.bi_off + x), __ldg(T.bi_off + x + 1), T.nb8, [&](int tok) { return cand_maybe(set, tok) ? cand_find(set, tok) : -1; }, fj == lane ? t : -1, lane,
                                [&](int j, uint32_t pay, uint32_t) { out[j] = __uint_as_float(pay); });
    __syncwarp();
    if (lane < k && fj != lane) out[lane] = out[fj];     // a repeated token takes its first position's score
  } else {
    uint2* out = cx + (i == 0 ? 1 : 1 + k + (i - 1) * k * k + jb * k);
    if (lane < k) out[lane] = make_uint2(0u, 0u);
    __syncwarp();
    if (have)
      warp_list_match<16>(T.tri_node, __ldg(T.tri_off + x), __ldg(T.tri_off + x + 1), T.nb8, [&](int tok) { return cand_maybe(set, tok) ? cand_find(set, tok) : -1; }, fj == lane ? t : -1, lane,
                                [&](int j, uint32_t pay, uint32_t idx) {
                                  out[j] = make_uint2(pay, __ldg(&T.tri_node[idx + 1]).y);
                                });
    __syncwarp();
    if (lane < k && fj != lane) out[lane] = out[fj];
  }
}

// The tree kernel of the trie layout.
// MAXT: launch bound (512 leaves the compiler twice the registers; 1024 covers beam * topk up to 1024)
// TRIE: always true here (the hash layout runs tree_hash_kernel below); the N-gram is the child-list trie
// (3-gram scores: search the context's children, located by the sweep).
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
  const int ctx1 = p.ctx_tail[2 * b + 1];
  const float* bg = p.bg + (size_t)b * sweep_bigrams(k, p.n_levels);  // bigram scores from the sweep kernel
  const uint2* cx = TRIE ? p.cx + (size_t)b * sweep_contexts(k, p.n_levels) : nullptr;

  if (tid == 0) {
    m.n_score[0] = 0.f; m.n_clamp[0] = INFINITY; m.n_tok[0] = ctx1; m.n_par[0] = -1; m.n_j[0] = 0;
    m.beam_a[0] = 0; m.lvl_base[0] = 1;
  }
  if (TRIE) {   // candidate sets of all levels: warp l builds level l's (l, l + warps, ...)
    const int nwarp = nthr >> 5;
    for (int l = warp; l < L; l += nwarp) {
      cand_clear(m.sets[l], lane);
      __syncwarp();
      const int t = lane < k ? ids[l * k + lane] : -1;
      if (t >= 0) cand_insert(m.sets[l], t, lane);
      __syncwarp();
      if (lane < k) m.fj[l * k + lane] = (unsigned char)(t >= 0 ? cand_find(m.sets[l], t) : lane);
    }
    for (int e = tid; e < 64; e += nthr) m.hit[e] = 0u;
    if (tid == 0) m.cxs[0] = __ldg(cx);   // level 0's only context
    __syncthreads();
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
    uint32_t* s3 = m.s3 + (i & 1) * w * k;
    uint32_t* hit = m.hit + (i & 1) * 32;
    // the ranges level i+1 can ask for, on their way to shared memory while this level is scored
    const int n_pre = !TRIE || i + 1 >= L ? 0 : i == 0 ? k : k * k;
    const uint2* pre_src = TRIE ? cx + (i == 0 ? 1 : 1 + k + (i - 1) * k * k) : nullptr;
    uint2 pre0 = make_uint2(0u, 0u), pre1 = pre0;
    if (tid < n_pre) pre0 = __ldg(pre_src + tid);
    if (tid + nthr < n_pre) pre1 = __ldg(pre_src + tid + nthr);
    if (TRIE) {   // one warp per beam entry: the children of its context, located by the sweep, against S_i
      const int nwarp = nthr >> 5;
      const uint2* cxs = m.cxs + (i & 1) * k * k;
      for (int rho = warp; rho < nb; rho += nwarp) {
        const int node = beam[rho], jn = m.n_j[node];
        const uint2 range = cxs[i == 0 ? 0 : i == 1 ? jn : (int)m.n_j[m.n_par[node]] * k + jn];
        const int my_t = (lane < k && m.fj[i * k + lane] == lane) ? ids[i * k + lane] : -1;
        warp_list_match<16>(p.trie.tri_ent, range.x, range.y, p.trie.nb8, [&](int tok) { return cand_maybe(m.sets[i], tok) ? cand_find(m.sets[i], tok) : -1; }, my_t, lane, [&](int j, uint32_t pay, uint32_t) {
          s3[rho * k + j] = pay;
          atomicOr(&hit[rho], 1u << j);
        });
      }
      __syncthreads();
    }
    if (tid < ncand) {
      const int rho = tid / k, j = tid - rho * k;
      const int node = beam[rho];
      const int t = ids[i * k + j];
      float s_ng = __ldg(bg + (i == 0 ? j : k + (i - 1) * k * k + (int)m.n_j[node] * k + j));
      if (TRIE) {
        const int f = m.fj[i * k + j];
        if ((hit[rho] >> f) & 1u) s_ng = __uint_as_float(s3[rho * k + f]);
      }
      const float inc = __fmul_rn(__fadd_rn(__fmul_rn(p.wl[i], sl[i * k + j]), __fmul_rn(p.wn, s_ng)), p.wv[i]);
      s = __fadd_rn(m.n_score[node], inc);
      const float pc = m.n_clamp[node];
      cl = s < pc ? s : pc;
      const int n = base + tid;
      m.n_score[n] = s; m.n_clamp[n] = cl; m.n_tok[n] = t; m.n_par[n] = node; m.n_j[n] = (unsigned char)j;
    }
    if (TRIE) {
      if (tid < 32) m.hit[((i + 1) & 1) * 32 + tid] = 0u;   // the next level's masks (read two barriers from now)
      uint2* nxt = m.cxs + ((i + 1) & 1) * k * k;
      if (tid < n_pre) nxt[tid] = pre0;
      if (tid + nthr < n_pre) nxt[tid + nthr] = pre1;
      for (int e = tid + 2 * nthr; e < n_pre; e += nthr) nxt[e] = __ldg(pre_src + e);
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


// ------------------------------------------------------------------------------------------------------
// The tree kernel of the hash layout: Algorithm 1 over the dense score table of ngram_sweep_kernel.
// ------------------------------------------------------------------------------------------------------
struct HashTreeSmem {
  float* n_score; float* n_clamp; int* n_tok; int* n_par; unsigned char* n_j;   // per node (the root is node 0); n_j: its candidate index
  int* c_ids; float* c_sl;                         // [L][k] the candidates' ids and s_logit, staged once
  int* b_node; float* b_sc; float* b_cl; int* b_row; int* b_bg;   // per beam entry: node, score, clamped score, rows of its context in the level's 3-gram and 2-gram tables
  Key* lvl_sorted;                                 // [2][64] best of a level by clamped score (the running best lags one level behind)
  int* sel; int* par_out; int* lvl_base;
  SelectSmem* ss;
  float* sg01; float* slice;                       // staged score tables: the small ones; one level's slice of t3
};
__host__ __device__ inline size_t hash_tree_layout(int k, int w, int budget, int L, bool stage, unsigned char* base, HashTreeSmem* t) {
  const int n_max = 1 + k + (L - 1) * w * k;
  const SgLayout g = sg_layout(k, L);
  size_t o = 0;
  auto take = [&](size_t bytes) { const size_t r = o; o += (bytes + 15) & ~size_t(15); return r; };
  const size_t o_sc = take((size_t)n_max * 4), o_cl = take((size_t)n_max * 4), o_tok = take((size_t)n_max * 4), o_par = take((size_t)n_max * 4),
               o_nj = take((size_t)n_max),
               o_ci = take((size_t)L * k * 4), o_cs = take((size_t)L * k * 4),
               o_bn = take((size_t)w * 4), o_bs = take((size_t)w * 4), o_bc = take((size_t)w * 4), o_br = take((size_t)w * 4), o_bb = take((size_t)w * 4),
               o_ls = take(2 * 64 * 8), o_sel = take((size_t)(budget + 1) * 4), o_po = take((size_t)budget * 4),
               o_lb = take((size_t)(L + 1) * 4), o_ss = take(sizeof(SelectSmem)),
               o_01 = take(stage ? (size_t)g.small * 4 : 0), o_sl = take(stage && L > 2 ? (size_t)g.st3 * 4 : 0);
  if (t != nullptr) {
    t->n_score = reinterpret_cast<float*>(base + o_sc);
    t->n_clamp = reinterpret_cast<float*>(base + o_cl); t->n_tok = reinterpret_cast<int*>(base + o_tok);
    t->n_par = reinterpret_cast<int*>(base + o_par); t->n_j = base + o_nj;
    t->c_ids = reinterpret_cast<int*>(base + o_ci); t->c_sl = reinterpret_cast<float*>(base + o_cs);
    t->b_node = reinterpret_cast<int*>(base + o_bn); t->b_sc = reinterpret_cast<float*>(base + o_bs);
    t->b_cl = reinterpret_cast<float*>(base + o_bc); t->b_row = reinterpret_cast<int*>(base + o_br); t->b_bg = reinterpret_cast<int*>(base + o_bb);
    t->lvl_sorted = reinterpret_cast<Key*>(base + o_ls);
    t->sel = reinterpret_cast<int*>(base + o_sel); t->par_out = reinterpret_cast<int*>(base + o_po);
    t->lvl_base = reinterpret_cast<int*>(base + o_lb); t->ss = reinterpret_cast<SelectSmem*>(base + o_ss);
    t->sg01 = reinterpret_cast<float*>(base + o_01); t->slice = reinterpret_cast<float*>(base + o_sl);
  }
  return o;
}

// 16-byte asynchronous copies global -> shared by the whole block (n4 chunks), one commit group.
__device__ __forceinline__ void copy_async16(float* dst, const float* src, int n4) {
  for (int e = threadIdx.x; e < n4; e += blockDim.x) {
    const unsigned d = (unsigned)__cvta_generic_to_shared(dst + 4 * e);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(src + 4 * e) : "memory");
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
}

// STAGE: the score table's slices are staged in shared memory (they fit for the paper's k = 25); otherwise the
// level loop reads the table where the sweep left it (L2).
template <int MAXT, bool STAGE>
__global__ void __launch_bounds__(MAXT) tree_hash_kernel(const TreeParams p) {
  extern __shared__ __align__(16) unsigned char tsm[];
  const int k = p.topk, w = p.beam, theta = p.budget - 1;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthr = blockDim.x, last_warp = (nthr >> 5) - 1;
  const SgLayout g = sg_layout(k, p.n_levels);
  const int b = blockIdx.x;
  const int fr = p.first_rows[b], L = min(p.n_levels, p.K - fr);   // this sequence's level 0 row and levels
  // When the block has a warp beyond the candidates (the launch adds one where 1024 threads allow it), that warp takes
  // no part in the selection: it keeps the running best 64, merging one level behind while the others select.
  const bool spare = w * k <= nthr - 32 && p.budget <= nthr - 32 && nthr >= 128;
  const bool idle = spare && warp == last_warp;
  const int n_active = spare ? nthr - 32 : nthr;
  const int my_rho = tid / k, my_j = tid - my_rho * k;              // this thread's (beam entry, candidate) pair at every level
  HashTreeSmem m;
  hash_tree_layout(k, w, p.budget, p.n_levels, STAGE, tsm, &m);
  __shared__ unsigned long long s_bits[64];
#ifdef DART_TREE_TL
  __shared__ long long s_tl[40];
  int n_tl = 0;
  const long long tl0 = clock64();
#define TL_STAMP() do { if (tid == 0 && n_tl < 40) s_tl[n_tl] = clock64() - tl0; ++n_tl; } while (0)
#else
#define TL_STAMP() do {} while (0)
#endif

  if (tid == 0) { m.n_score[0] = 0.f; m.n_clamp[0] = INFINITY; m.n_par[0] = -1; m.n_j[0] = 0; m.b_node[0] = 0; m.b_sc[0] = 0.f; m.b_cl[0] = INFINITY; m.b_row[0] = 0; m.b_bg[0] = 0; m.lvl_base[0] = 1; }
  pdl_wait();
  TL_STAMP();
  const int* ids = p.ids + ((size_t)b * p.K + fr) * k;
  const float* sl = p.slogit + ((size_t)b * p.K + fr) * k;
  const float* sg = p.sg + (size_t)b * g.total;
  if (tid == 0) m.n_tok[0] = p.ctx_tail[2 * b + 1];
  for (int e = tid; e < L * k; e += nthr) { m.c_ids[e] = ids[e]; m.c_sl[e] = sl[e]; }
  if (STAGE) {
    copy_async16(m.sg01, sg, g.small / 4);
    asm volatile("cp.async.wait_all;" ::: "memory");    // the small tables
  }
  block_select_init(m.ss);
  __syncthreads();
  // running best 64 by (clamped score desc, node index asc): lives in the last warp's registers
  Key g0 = kPadKey, g1 = kPadKey;
  TL_STAMP();

  int nb = 1;
  for (int i = 0; i < L; ++i) {
    const int ncand = nb * k;
    const int base = m.lvl_base[i];
    float s = -INFINITY, cl = -INFINITY;
    if (tid < ncand) {
      const int rho = my_rho, j = my_j;
      const int t = m.c_ids[i * k + j];
      // the candidate's 3-gram entry, or -- no such row -- its 2-gram entry
      const int at3 = (i == 0 ? g.t0 : i == 1 ? g.t1 : g.small + (i - 2) * g.st3) + m.b_row[rho] + j;
      const int at2 = (i == 0 ? 0 : g.bg + (i - 1) * k * k) + m.b_bg[rho] + j;
      float s3, s2;
      if (STAGE) { s3 = i < 2 ? m.sg01[at3] : m.slice[at3 - g.small - (i - 2) * g.st3]; s2 = m.sg01[at2]; }
      else { s3 = __ldg(sg + at3); s2 = __ldg(sg + at2); }
      const float s_ng = __float_as_uint(s3) == kNoRowBits ? s2 : s3;
      const float inc = __fmul_rn(__fadd_rn(__fmul_rn(p.wl[i], m.c_sl[i * k + j]), __fmul_rn(p.wn, s_ng)), p.wv[i]);
      s = __fadd_rn(m.b_sc[rho], inc);
      const float pc = m.b_cl[rho];
      cl = s < pc ? s : pc;
      const int n = base + tid;
      DART_CHECK(n < 1 + k + (p.n_levels - 1) * w * k, p.status) {   // inside the node arrays
        m.n_score[n] = s; m.n_clamp[n] = cl; m.n_tok[n] = t; m.n_par[n] = m.b_node[rho]; m.n_j[n] = (unsigned char)j;
      }
    }
    // keys carry the node index base + tid, which orders candidates of one level like tid does
    // best 64 by score -> next beam; `differs`: some clamped score is not its score (never, when increments <= 0)
    TL_STAMP();
    const int fetch = i == 0 ? (L > 2 ? 2 : -1) : ((i >= 2 && i + 1 < L) ? i + 1 : -1);   // the level whose slice is fetched while this one is selected
    const int nb_next = ncand < w ? ncand : w;
    Key* lvl_out = m.lvl_sorted + (i & 1) * 64;
    const int differs = block_select64(
        tid < ncand ? make_key(s, base + tid) : kPadKey, s, tid < ncand && cl != s, idle, n_active, m.ss,
        [&](int r, Key key, int any) {
          DART_CHECK(r >= 0 && r < 64, p.status)
          if (!any) lvl_out[r] = key;
          if (r < nb_next) {
            // beam entry r of the next level: its node, scores and the row of its context -- (the parent's candidate
            // index, this node's candidate index) -- in the next level's slice of the score table
            const int node = key_index(key), j = m.n_j[node];
            m.b_node[r] = node;
            m.b_sc[r] = m.n_score[node];
            m.b_cl[r] = m.n_clamp[node];
            m.b_row[r] = (i == 0 ? j : (int)m.n_j[m.n_par[node]] * k + j) * k;
            m.b_bg[r] = j * k;
          }
        },
        [&]() {
          // every thread has read what it needs of level i's slice: the next one may overwrite it (levels 0 and 1 use
          // the small table, so level 2's slice is fetched during level 0 and nothing during level 1)
          if (STAGE && fetch >= 0) copy_async16(m.slice, sg + g.small + (fetch - 2) * g.st3, g.st3 / 4);
          if (idle && i > 0) {   // the spare warp: the running best takes in the previous level's best 64
            const Key* q = m.lvl_sorted + ((i - 1) & 1) * 64;
            merge_keep64(g0, g1, q[lane], q[32 + lane], lane);
          }
        },
        [&]() {
          // without a spare warp the last warp does that while the first warps rank this level's survivors
          if (!spare && warp == last_warp && i > 0) {
            const Key* q = m.lvl_sorted + ((i - 1) & 1) * 64;
            merge_keep64(g0, g1, q[lane], q[32 + lane], lane);
          }
          if (tid == 0) m.lvl_base[i + 1] = base + ncand;
          if (STAGE && i >= 1) asm volatile("cp.async.wait_all;" ::: "memory");   // the next level's slice has landed
        });
    if (differs)   // the level's best 64 by clamped score are a different set: select again
      block_select64(tid < ncand ? make_key(cl, base + tid) : kPadKey, cl, 0, idle, n_active, m.ss, [&](int r, Key key, int) { lvl_out[r] = key; }, [] {}, [] {});
    TL_STAMP();
    nb = nb_next;
  }
  if (warp == last_warp && L > 0) {
    const Key* q = m.lvl_sorted + ((L - 1) & 1) * 64;
    merge_keep64(g0, g1, q[lane], q[32 + lane], lane);
  }

  // ---- the selected nodes: the first n_sel entries of the running best 64; slot_of: node -> output slot
  const int total = m.lvl_base[L] - 1;
  const int n_sel = total < theta ? total : theta;
  int* slot_of = reinterpret_cast<int*>(m.n_score);   // the scores are no longer needed
  if (warp == last_warp) {
    if (lane < n_sel) { const int n = key_index(g0); m.sel[1 + lane] = n; slot_of[n] = 1 + lane; }
    if (32 + lane < n_sel) { const int n = key_index(g1); m.sel[33 + lane] = n; slot_of[n] = 33 + lane; }
    if (lane == 0) { m.sel[0] = 0; slot_of[0] = 0; }
  }
  __syncthreads();
  // the selection is closed under "parent of" (clamped scores never rise along a path), so every parent has a slot
  const int budget = p.budget;
  for (int x = tid; x < budget; x += nthr) m.par_out[x] = (x >= 1 && x <= n_sel) ? slot_of[m.n_par[m.sel[x]]] : -1;
  __syncthreads();
  for (int x = tid; x < budget; x += nthr) {
    const size_t o = (size_t)b * budget + x;
    unsigned long long bits = 0ull;
    if (x <= n_sel) {
      const int n = m.sel[x];
      int y = x;
      for (int guard = 0; guard <= L + 1 && y >= 0; ++guard) { bits |= 1ull << y; y = m.par_out[y]; }
      p.tokens[o] = m.n_tok[n];
      p.parents[o] = m.par_out[x];
      p.depth[o] = __popcll(bits) - 1;                 // a node's depth = its ancestors, the root (depth 0) among them
      if (p.scores) p.scores[o] = x == 0 ? 0.f : m.n_clamp[n];
    } else {
      p.tokens[o] = -1; p.parents[o] = -1; p.depth[o] = -1;
      if (p.scores) p.scores[o] = -INFINITY;
    }
    s_bits[x] = bits;
  }
  if (tid == 0) p.n_nodes[b] = 1 + n_sel;
  __syncthreads();
  uint8_t* mbase = p.mask + (size_t)b * budget * budget;
  for (int x = warp; x < budget; x += nthr >> 5) {      // a warp per row of the mask
    const unsigned long long bits = s_bits[x];
    for (int y = lane; y < budget; y += 32) mbase[x * budget + y] = (uint8_t)((bits >> y) & 1ull);
  }
#ifdef DART_TREE_TL
  TL_STAMP();
  __syncthreads();
  if (tid == 0 && p.scores)
  {
    for (int e = 0; e < n_tl && e < 40 && 1 + e < budget; ++e) p.scores[(size_t)b * budget + 1 + e] = (float)s_tl[e];
    for (int e = 0; e < 11 && 45 + e < budget; ++e) p.scores[(size_t)b * budget + 45 + e] = (float)g_sel_tl[e];
  }
#endif
#undef TL_STAMP
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
// The hash-layout kernel stages the score table's slices in shared memory when they fit beside the nodes.
constexpr size_t kTreeSmemMax = 200 * 1024;
static bool hash_tree_stages(int topk, int beam, int budget, int n_levels) {
  return hash_tree_layout(topk, beam, budget, n_levels, true, nullptr, nullptr) + 16 <= kTreeSmemMax;
}
static size_t hash_tree_smem_bytes(int topk, int beam, int budget, int n_levels) {
  return hash_tree_layout(topk, beam, budget, n_levels, hash_tree_stages(topk, beam, budget, n_levels), nullptr, nullptr) + 16;
}

template <class K>
static cudaError_t allow_smem(K kernel, size_t smem) {
  return smem > 48 * 1024 ? cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) : cudaSuccess;
}

cudaError_t tree_setup(int topk, int beam, int budget, int max_levels) {
  size_t smem = tree_smem_bytes(topk, beam, budget, max_levels);
  cudaError_t e = allow_smem(tree_kernel<512, true>, smem);
  if (e == cudaSuccess) e = allow_smem(tree_kernel<1024, true>, smem);
  smem = hash_tree_smem_bytes(topk, beam, budget, max_levels);
  if (e == cudaSuccess) e = allow_smem(tree_hash_kernel<576, true>, smem);
  if (e == cudaSuccess) e = allow_smem(tree_hash_kernel<1024, true>, smem);
  if (e == cudaSuccess) e = allow_smem(tree_hash_kernel<576, false>, smem);
  if (e == cudaSuccess) e = allow_smem(tree_hash_kernel<1024, false>, smem);
  return e;
}

template <bool STAGE>
static cudaError_t launch_hash_tree(const TreeParams& p, int threads, size_t smem, cudaStream_t st) {
  if (threads <= 576) return launch_pdl(tree_hash_kernel<576, STAGE>, dim3(p.B), dim3(threads), smem, st, p);
  return launch_pdl(tree_hash_kernel<1024, STAGE>, dim3(p.B), dim3(threads), smem, st, p);
}

cudaError_t launch_tree(const TreeParams& p, cudaStream_t st) {
  const bool trie = p.trie.bi_off != nullptr;
  // one thread per (beam entry, candidate) pair; a smaller block makes every barrier cheaper
  int need = p.beam * p.topk;
  if (p.budget > need) need = p.budget;
  if (need < 64) need = 64;
  if (trie && 32 * p.beam > need) need = 32 * p.beam;   // one warp per beam entry reads its context's children
  int threads = (need + 31) / 32 * 32;
  if (threads > 1024) threads = 1024;
  if (!trie && threads + 32 <= 1024) threads += 32;     // a spare warp that keeps the running best (see tree_hash_kernel)
  if (trie) {
    const int n_task = p.n_levels * 2 * p.topk;   // one warp per (level, list kind, context position)
    const cudaError_t e = launch_pdl(trie_sweep_kernel, dim3((n_task + 7) / 8, p.B), dim3(256), 0, st, p);
    if (e != cudaSuccess) return e;
    const size_t smem = tree_smem_bytes(p.topk, p.beam, p.budget, p.n_levels);
    if (threads <= 512) return launch_pdl(tree_kernel<512, true>, dim3(p.B), dim3(threads), smem, st, p);
    return launch_pdl(tree_kernel<1024, true>, dim3(p.B), dim3(threads), smem, st, p);
  }
  // (Sweep and tree as one launch -- sweep blocks that count themselves done, a tree block that waits for the count of a
  // slice before fetching it -- was built and measured slower, 41.7 against 35.8 us at the 14B shape: the fence, the
  // count and the poll cost more than the launch they replace.)
  const int n3 = p.n_levels > 2 ? p.n_levels - 2 : 0;
  const int n_rows = sweep_small_rows(p.topk, p.n_levels) + n3 * p.topk * p.topk;
  const cudaError_t e = launch_pdl(ngram_sweep_kernel, dim3((n_rows + 7) / 8, p.B), dim3(256), 0, st, p);
  if (e != cudaSuccess) return e;
  const bool stage = hash_tree_stages(p.topk, p.beam, p.budget, p.n_levels);
  const size_t smem = hash_tree_layout(p.topk, p.beam, p.budget, p.n_levels, stage, nullptr, nullptr) + 16;
  return stage ? launch_hash_tree<true>(p, threads, smem, st) : launch_hash_tree<false>(p, threads, smem, st);
}


}  // namespace dart
