// C ABI of the DART drafting step: handle management, argument validation, launch planning.
// Every arithmetic step of the path runs in the kernels of this directory; this file only
// validates, sizes and enqueues.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <vector>

#include "../../include/dart.h"
#include "kernels.h"

using namespace dart;

namespace {

int g_init_cuda_error = 0;

struct Workspace {
  void* base = nullptr;
  size_t bytes = 0;
  float* part = nullptr;        // split partials of the current projection
  float* res0 = nullptr;        // [max_batch*K, h]  g of the fresh rows (first residual)
  float* x1 = nullptr;          // [Mmax, h] residual stream after attention
  bf16 *z_hi = nullptr, *z_lo = nullptr;   // [Mmax, 2h]: z row of every token row (b, r); <mask> rows are copies of zmask
  bf16 *zmask_hi = nullptr, *zmask_lo = nullptr;   // [2h] the <mask> row, written once at init
  bf16 *q_hi = nullptr, *q_lo = nullptr;   // [Mmax, Hq*dh]
  bf16 *k_new = nullptr, *v_new = nullptr; // [max_batch, Hkv, 16, dh]
  bf16 *a_hi = nullptr, *a_lo = nullptr;   // [Mmax, Hq*dh]
  bf16 *n_hi = nullptr, *n_lo = nullptr;   // [Mmax, h]  gain-scaled residual (not yet divided by its rms)
  bf16 *u_hi = nullptr, *u_lo = nullptr;   // [Mmax, I]
  float *ss_g = nullptr, *ss_1 = nullptr, *ss_2 = nullptr;  // [h/128 tiles][MP] sums of squares per tile
  float* rstd_mask = nullptr;
  float* mask_res = nullptr;    // [h] g half of the <mask> representation as fp32
  float2* rope_tab = nullptr;   // [max_prefix + K][dh/2] (cos, sin)
  float* sg = nullptr;          // [max_batch][tree_sg_floats] dense N-gram scores of the tree builder (hash layout)
  float* bg = nullptr;          // [max_batch][topk + (K-1)*topk^2] bigram scores of the tree builder (trie layout)
  uint2* cx = nullptr;          // [max_batch][1 + topk + (K-2)*topk^2] child ranges of the 3-gram contexts (trie layout)
  float *o_part = nullptr, *ml_part = nullptr;
  float *lm_stats = nullptr, *lm_key = nullptr, *lm_y = nullptr;
  int32_t* lm_id = nullptr;
  int* status = nullptr;
  bf16* pz = nullptr;           // prefill: z of one pass [kPrefillPassRows, 2h] bf16
  float* pss = nullptr;         // prefill: per-row partial sums of squares of g [kPrefillPassRows, h/256]
  float* lm_pieces = nullptr;   // [SMs][128][MPmax] partial logits of vocabulary tiles cut between CTAs
  int* lm_flags = nullptr;      // [SMs] launch tag of each CTA's piece
  unsigned long long* lm_bound = nullptr;   // [128][kLmBoundSlots] lower bounds the LM head's CTAs share (many token rows)
};

}  // namespace

namespace dart {
void record_global_cuda_error(cudaError_t e) { g_init_cuda_error = (int)e; }
}  // namespace dart

struct dart_handle {
  dart_config cfg;
  dart_weights w;
  int device = 0;
  int n_sm = 0;
  int last_cuda_error = 0;
  GemmPlan plan_fc, plan_qkv, plan_o, plan_gu, plan_down;
  UmmaMaps maps_fc, maps_qkv, maps_o, maps_gu, maps_down;
  // gate / up with row ownership where the shape suits it, at up to 8 [0], 32 [1] and 128 [2] token rows
  bool own_ok[3] = {false, false, false};
  OwnPlan own_gu[3];
  CUtensorMap own_w_gu[3][2];
  CUtensorMap pmap_fc, pmap_kv[4];   // prefill: W_fc, and the g-/e-half columns of W_k and W_v (boxes of 256 rows)
  CUtensorMap map_lm;        // the LM head's weight matrix (boxes of 128 rows)
  CUtensorMap map_lm256;     // the same with boxes of 256 rows, for the swapped-operand kernel (33..128 token rows)
  CUtensorMap lmx_hi, lmx_lo; int lmx_M = -1;   // that kernel's activation maps [M][h], boxes of 128 rows
  int lm_tag = 0;            // launch counter of the LM head (marks its cross-CTA pieces)
  int maps_M = -1;           // token rows the activation tensor maps were encoded for
  const void* maps_feats = nullptr; int maps_fc_M = -1;
  int lm_grid = 0;
  int attn_pairs_cap = 0;  // capacity of the attention partial buffers in (sequence, chunk) pairs
  AttnUmmaMaps attn_maps;  // q and new-row maps encoded at init; cache maps follow the caller's pointers
  const void* attn_k_ptr = nullptr;
  const void* attn_v_ptr = nullptr;
  int h_tiles = 0;         // 128-row tiles of a hidden-sized row
  Workspace ws;
  void* ng_base = nullptr;       // the hash layout's allocation: fingerprint words, then slots
  NgramSlot* ng_slots = nullptr;
  uint32_t ng_mask = 0, ng_max_probe = 0;
  NgramTrieOwned ng_trie{};     // the child-list layout (ngram_layout = DART_NGRAM_TRIE)
  size_t ng_bytes = 0;
  float wl[8], wv[8], wn, miss;
  std::vector<void*> owned;  // small device arrays (plan tables, counters)
  int z_B = -1;              // row pattern (batch, per-sequence fresh rows) the <mask> rows of z were last written for
  FreshOffsets z_foff = {};
  int prof_stage = -1;       // measurement aid: stage whose kernels the next call brackets with events
  cudaEvent_t prof_start = nullptr, prof_stop = nullptr;
};

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
bool aligned16(const void* p) { return p != nullptr && (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool aligned32(const void* p) { return p != nullptr && (reinterpret_cast<uintptr_t>(p) & 31u) == 0; }

bool config_ok(const dart_config* c) {
  if (c == nullptr || c->struct_size != sizeof(dart_config)) return false;
  if (c->hidden < 64 || c->hidden % 64 != 0) return false;
  if (c->head_dim != 64 && c->head_dim != 128) return false;
  if (c->n_q_heads < 1 || c->n_kv_heads < 1 || c->n_q_heads % c->n_kv_heads != 0) return false;
  if (c->K < 1 || c->K > 8) return false;
  if ((c->n_q_heads / c->n_kv_heads) * c->K > 64) return false;
  if (c->mlp_inter < 16 || c->mlp_inter % 16 != 0) return false;
  if (c->vocab < 16 || c->vocab % 16 != 0 || c->vocab >= (1 << 21) - 1) return false;
  if (c->feat_in != 0 && (c->feat_in < 16 || c->feat_in % 16 != 0)) return false;   // 0: the caller passes g itself
  if (c->max_batch < 1 || c->max_batch > 32 || c->max_batch * c->K > 128) return false;
  if (c->max_prefix < 1) return false;
  if (c->topk < 1 || c->topk > 32 || c->topk > c->vocab) return false;
  if (c->beam < 1 || c->beam > 32) return false;
  if (c->tree_budget < 2 || c->tree_budget > 64) return false;
  if (c->ngram_order != 2 && c->ngram_order != 3) return false;
  if (c->ngram_layout != DART_NGRAM_HASH && c->ngram_layout != DART_NGRAM_TRIE) return false;
  if (!(c->rope_theta > 0.f) || !(c->rms_eps >= 0.f) || !(c->temperature >= 0.f)) return false;
  if (!(c->eps_ng > 0.f) || !(c->eps_logit >= 0.f)) return false;
  return true;
}

struct PlanHost {
  GemmPlan plan;
  std::vector<int> expected, meta;
};

// Cut the flattened (128-row tile, 64-k block) space of a projection into `grid_target` equal ranges, one
// persistent CTA per SM; a CTA's piece of a tile holds all 128 rows.  The piece table keeps the 16-row
// granularity of the fused finalize: the j-th 16 rows of a 128-row piece at slot s are "piece" 8 s + j.
void make_plan_host(PlanHost& ph, const GemmSeg* segs, int nseg, int Kd, int grid_target, int pair_offset) {
  GemmPlan& p = ph.plan;
  memset(&p, 0, sizeof(p));
  p.nseg = nseg;
  int tiles = 0;
  for (int i = 0; i < 6; ++i) {
    if (i < nseg) {
      p.seg[i] = segs[i];
      p.seg[i].tile0 = tiles;
      tiles += (segs[i].rows + 127) / 128;
    } else {
      p.seg[i] = p.seg[0];
    }
  }
  p.Kd = Kd;
  p.SK = (Kd + 63) / 64;
  p.KR = (p.SK + kUmmaKS - 1) / kUmmaKS;   // a work unit = one ring stage = kUmmaKS k-blocks (a k tail reads as zeros)
  p.n_tiles = tiles;
  p.U = (long long)tiles * p.KR;
  p.grid = (int)((long long)grid_target < p.U ? grid_target : p.U);
  while (p.grid > 1 && (p.KR + (p.U / p.grid) - 1) / (p.U / p.grid) + 1 > kMetaStride - 1) p.grid /= 2;
  p.pair_offset = pair_offset;
  p.n_groups = pair_offset > 0 ? pair_offset : tiles;
  p.slots = 1;
  p.meta_stride = kMetaStride;
  ph.expected.assign(p.n_groups, 0);
  ph.meta.assign((size_t)tiles * 8 * kMetaStride, 0);
  for (int c = 0; c < p.grid; ++c) {
    const long long u0 = ((long long)c * p.U) / p.grid, u1 = ((long long)(c + 1) * p.U) / p.grid;
    if (u0 >= u1) continue;
    const int t0 = (int)(u0 / p.KR), t1 = (int)((u1 - 1) / p.KR);
    if (t1 - t0 + 1 > p.slots) p.slots = t1 - t0 + 1;
  }
  for (int c = 0; c < p.grid; ++c) {
    const long long u0 = ((long long)c * p.U) / p.grid, u1 = ((long long)(c + 1) * p.U) / p.grid;
    if (u0 >= u1) continue;
    const int t0 = (int)(u0 / p.KR), t1 = (int)((u1 - 1) / p.KR);
    for (int t = t0; t <= t1; ++t) {
      // t counts tiles in unit order: paired tiles alternate (T, T + pair_offset, T + 1, ...), see umma_gemm.cu
      const int T = pair_offset > 0 ? (t & 1) * pair_offset + (t >> 1) : t;
      ph.expected[pair_offset > 0 ? t >> 1 : t] += 1;
      for (int j = 0; j < 8; ++j) {
        int& n = ph.meta[(size_t)(T * 8 + j) * kMetaStride];
        if (n < kMetaStride - 1) ph.meta[(size_t)(T * 8 + j) * kMetaStride + 1 + n++] = (c * p.slots + (t - t0)) * 8 + j;
      }
    }
  }
}

size_t part_floats(const GemmPlan& p, int MP) { return (size_t)p.grid * p.slots * 128 * MP; }

struct Layout {
  size_t total = 0;
  size_t take(size_t bytes) {
    const size_t off = total;
    total += align_up(bytes, 256);
    return off;
  }
};

// Token rows the workspace is sized for.
int token_rows_capacity(const dart_config& c) { return c.max_batch * c.K; }
// Rows one pass of the draft-side prefill handles (its z and sums-of-squares buffers are sized for this).
constexpr int kPrefillPassRows = 4096;
int prefill_fc_tiles(const dart_config& c) { return (c.hidden + 255) / 256; }

// Sizes every workspace region; with base != nullptr also assigns the pointers.
size_t layout_workspace(const dart_config& c, size_t part_max_floats, int attn_pairs_cap, int lm_grid, char* base, Workspace* ws) {
  Layout L;
  const size_t Mmax = (size_t)token_rows_capacity(c);
  const size_t MPmax = padded_tokens((int)Mmax);
  const size_t dq = (size_t)c.n_q_heads * c.head_dim;
  const size_t ht = (c.hidden + 127) / 128;
  size_t o;
#define TAKE(field, type, bytes) \
  o = L.take(bytes);             \
  if (base) ws->field = reinterpret_cast<type>(base + o);
  TAKE(part, float*, part_max_floats * sizeof(float));
  TAKE(res0, float*, Mmax * c.hidden * sizeof(float));
  TAKE(x1, float*, Mmax * c.hidden * sizeof(float));
  TAKE(z_hi, bf16*, Mmax * 2 * c.hidden * sizeof(bf16));
  TAKE(z_lo, bf16*, Mmax * 2 * c.hidden * sizeof(bf16));
  TAKE(zmask_hi, bf16*, (size_t)2 * c.hidden * sizeof(bf16));
  TAKE(zmask_lo, bf16*, (size_t)2 * c.hidden * sizeof(bf16));
  TAKE(q_hi, bf16*, Mmax * dq * sizeof(bf16));
  TAKE(q_lo, bf16*, Mmax * dq * sizeof(bf16));
  TAKE(k_new, bf16*, (size_t)c.max_batch * c.n_kv_heads * 16 * c.head_dim * sizeof(bf16));
  TAKE(v_new, bf16*, (size_t)c.max_batch * c.n_kv_heads * 16 * c.head_dim * sizeof(bf16));
  TAKE(a_hi, bf16*, Mmax * dq * sizeof(bf16));
  TAKE(a_lo, bf16*, Mmax * dq * sizeof(bf16));
  TAKE(n_hi, bf16*, Mmax * c.hidden * sizeof(bf16));
  TAKE(n_lo, bf16*, Mmax * c.hidden * sizeof(bf16));
  TAKE(u_hi, bf16*, Mmax * c.mlp_inter * sizeof(bf16));
  TAKE(u_lo, bf16*, Mmax * c.mlp_inter * sizeof(bf16));
  TAKE(ss_g, float*, ht * MPmax * sizeof(float));
  TAKE(ss_1, float*, ht * MPmax * sizeof(float));
  TAKE(ss_2, float*, ht * MPmax * sizeof(float));
  TAKE(rstd_mask, float*, 256);
  TAKE(mask_res, float*, (size_t)c.hidden * sizeof(float));
  TAKE(rope_tab, float2*, (size_t)(c.max_prefix + c.K) * (c.head_dim / 2) * sizeof(float2));
  TAKE(sg, float*, (size_t)c.max_batch * tree_sg_floats(c.topk, c.K) * sizeof(float));
  TAKE(bg, float*, (size_t)c.max_batch * (c.topk + (size_t)(c.K - 1) * c.topk * c.topk) * sizeof(float));
  TAKE(cx, uint2*, (size_t)c.max_batch * (1 + c.topk + (size_t)(c.K > 2 ? c.K - 2 : 0) * c.topk * c.topk) * sizeof(uint2));
  TAKE(o_part, float*, (size_t)attn_pairs_cap * c.n_kv_heads * 64 * c.head_dim * sizeof(float));
  TAKE(ml_part, float*, (size_t)attn_pairs_cap * c.n_kv_heads * 64 * 2 * sizeof(float));
  TAKE(lm_pieces, float*, (size_t)lm_grid * 128 * MPmax * sizeof(float));
  TAKE(lm_flags, int*, (size_t)lm_grid * sizeof(int));
  TAKE(lm_bound, unsigned long long*, (size_t)128 * kLmBoundSlots * sizeof(unsigned long long));
  TAKE(lm_stats, float*, (size_t)lm_grid * MPmax * 2 * sizeof(float));
  TAKE(lm_key, float*, (size_t)lm_grid * MPmax * 32 * sizeof(float));
  TAKE(lm_y, float*, (size_t)lm_grid * MPmax * 32 * sizeof(float));
  TAKE(lm_id, int32_t*, (size_t)lm_grid * MPmax * 32 * sizeof(int32_t));
  TAKE(status, int*, 256);
  if (c.feat_in > 0) {
    TAKE(pz, bf16*, (size_t)kPrefillPassRows * 2 * c.hidden * sizeof(bf16));
    TAKE(pss, float*, (size_t)kPrefillPassRows * prefill_fc_tiles(c) * sizeof(float));
  }
#undef TAKE
  return L.total;
}

struct PlanSet {
  PlanHost fc, qkv, o, gu, down;
  size_t part_max = 0;
};

void build_plans(const dart_config& c, const dart_weights* w, int n_sm, PlanSet& ps) {
  const int grid = n_sm;
  const int h = c.hidden, dq = c.n_q_heads * c.head_dim, dkv = c.n_kv_heads * c.head_dim;
  auto W = [&](const void* p, long long off) { return w ? static_cast<const bf16*>(p) + off : nullptr; };
  GemmSeg s[6];
  // without a feature FC (feat_in = 0) its plan is a stand-in over the first hidden columns of w_q, never launched
  s[0] = c.feat_in > 0 ? GemmSeg{W(w ? w->w_fc : nullptr, 0), h, 0, c.feat_in, 0} : GemmSeg{W(w ? w->w_q : nullptr, 0), h < dq ? h : dq, 0, 2 * h, 0};
  make_plan_host(ps.fc, s, 1, c.feat_in > 0 ? c.feat_in : h, grid, 0);
  // QKV reads z = [g-half | e-half] (2h wide); the two halves carry different 1/rms factors, so each
  // weight matrix is split into its g-half and e-half columns and the halves are finalized in pairs
  const int qt = (dq + 127) / 128, kt = (dkv + 127) / 128;
  s[0] = {W(w ? w->w_q : nullptr, 0), dq, 0, 2 * h, 0};
  s[1] = {W(w ? w->w_k : nullptr, 0), dkv, 0, 2 * h, 0};
  s[2] = {W(w ? w->w_v : nullptr, 0), dkv, 0, 2 * h, 0};
  s[3] = {W(w ? w->w_q : nullptr, h), dq, 0, 2 * h, h};
  s[4] = {W(w ? w->w_k : nullptr, h), dkv, 0, 2 * h, h};
  s[5] = {W(w ? w->w_v : nullptr, h), dkv, 0, 2 * h, h};
  make_plan_host(ps.qkv, s, 6, h, grid, qt + 2 * kt);
  s[0] = {W(w ? w->w_o : nullptr, 0), h, 0, dq, 0};
  make_plan_host(ps.o, s, 1, dq, grid, 0);
  s[0] = {W(w ? w->w_gate : nullptr, 0), c.mlp_inter, 0, h, 0};
  s[1] = {W(w ? w->w_up : nullptr, 0), c.mlp_inter, 0, h, 0};
  make_plan_host(ps.gu, s, 2, h, grid, (c.mlp_inter + 127) / 128);
  s[0] = {W(w ? w->w_down : nullptr, 0), h, 0, c.mlp_inter, 0};
  make_plan_host(ps.down, s, 1, c.mlp_inter, grid, 0);
  const int MPmax = padded_tokens(token_rows_capacity(c));
  const PlanHost* all[5] = {&ps.fc, &ps.qkv, &ps.o, &ps.gu, &ps.down};
  ps.part_max = 0;
  for (int i = 0; i < 5; ++i) {
    const size_t f = part_floats(all[i]->plan, MPmax);
    if (f > ps.part_max) ps.part_max = f;
  }
}

// Floats of the piece area: the largest projection's pieces at the largest token-row padding.
size_t part_capacity(const dart_config& c, int n_sm) {
  PlanSet a;
  build_plans(c, nullptr, n_sm, a);
  return a.part_max;
}

// Attention chunks of the one-chunk-per-CTA split: about two CTAs per SM, chunks of 128 .. 512 keys (longer chunks
// leave a CTA a long serial loop of 64-key tiles; measured at batch 16: 1792-key chunks 218 us, 448-key chunks 190 us).
// The tcgen05 split picks longer ones (attn_umma_chunk_keys), which need fewer partial slots than this bound.
constexpr int kAttnMaxChunk = 512;
int attn_pairs_capacity(const dart_config& c, int n_sm) {
  const long long by_sm = (2 * n_sm) / c.n_kv_heads, by_len = ((long long)c.max_batch * c.max_prefix + kAttnMaxChunk - 1) / kAttnMaxChunk;
  return (int)(by_sm > by_len ? by_sm : by_len) + 2 * c.max_batch + 2;
}

int fail_cuda(dart_handle* h, cudaError_t e) {
  if (h) h->last_cuda_error = (int)e; else g_init_cuda_error = (int)e;
  return DART_ERR_CUDA;
}

template <typename T>
cudaError_t upload(dart_handle* h, const std::vector<T>& v, T** out) {
  T* d = nullptr;
  const size_t nb = (v.size() ? v.size() : 1) * sizeof(T);
  cudaError_t e = cudaMalloc(&d, nb);
  if (e != cudaSuccess) return e;
  h->owned.push_back(d);
  if (v.size()) e = cudaMemcpy(d, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice);
  *out = d;
  return e;
}

}  // namespace

extern "C" {

const char* dart_status_string(int status) {
  switch (status) {
    case DART_OK: return "DART_OK";
    case DART_ERR_INVALID_ARG: return "DART_ERR_INVALID_ARG";
    case DART_ERR_UNSUPPORTED_ARCH: return "DART_ERR_UNSUPPORTED_ARCH";
    case DART_ERR_CUDA: return "DART_ERR_CUDA";
    case DART_ERR_CAPACITY: return "DART_ERR_CAPACITY";
    case DART_ERR_TIMEOUT: return "DART_ERR_TIMEOUT";
    case DART_ERR_INTERNAL: return "DART_ERR_INTERNAL";
    default: return "DART_ERR_UNKNOWN";
  }
}

size_t dart_workspace_bytes(const dart_config* cfg) {
  if (!config_ok(cfg)) return 0;
  const int n_sm = 148;  // sized for a B200; dart_draft_init uses the device's own count
  return layout_workspace(*cfg, part_capacity(*cfg, n_sm), attn_pairs_capacity(*cfg, n_sm), 2 * n_sm, nullptr, nullptr);
}

size_t dart_ngram_bytes(const dart_handle* h) { return h ? h->ng_bytes : 0; }

int dart_last_cuda_error(const dart_handle* h) { return h ? h->last_cuda_error : g_init_cuda_error; }

int dart_draft_init(const dart_config* cfg, const dart_weights* weights, const dart_ngram_host* ngram, dart_handle** out) {
  if (out == nullptr) return DART_ERR_INVALID_ARG;
  *out = nullptr;
  if (!config_ok(cfg) || weights == nullptr) return DART_ERR_INVALID_ARG;
  const void* wp[15] = {weights->w_fc, weights->embed, weights->mask_vec, weights->norm_g, weights->norm_e,
                        weights->w_q, weights->w_k, weights->w_v, weights->w_o, weights->norm_post,
                        weights->w_gate, weights->w_up, weights->w_down, weights->norm_final, weights->w_lm};
  for (int i = 0; i < 15; ++i)
    if (!aligned32(wp[i]) && !(i == 0 && cfg->feat_in == 0)) return DART_ERR_INVALID_ARG;  // the matrices are streamed with 32-byte loads
  if (ngram != nullptr && ngram->n_rows > 0 &&
      (ngram->order == nullptr || ngram->ctx0 == nullptr || ngram->ctx1 == nullptr || ngram->next == nullptr ||
       ngram->score == nullptr))
    return DART_ERR_INVALID_ARG;

  int dev = 0, major = 0, n_sm = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail_cuda(nullptr, e);
  e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  if (e != cudaSuccess) return fail_cuda(nullptr, e);
  if (major != 10) return DART_ERR_UNSUPPORTED_ARCH;
  e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return fail_cuda(nullptr, e);

  dart_handle* h = new dart_handle();
  h->cfg = *cfg;
  h->w = *weights;
  h->device = dev;
  h->n_sm = n_sm;
  h->h_tiles = (cfg->hidden + 127) / 128;

#define INIT_CHECK(expr)                                 \
  if ((e = (expr)) != cudaSuccess) {                     \
    g_init_cuda_error = (int)e;                          \
    dart_draft_destroy(h);                               \
    return DART_ERR_CUDA;                                \
  }

  {
    // every kernel of the path is fed by TMA: a driver whose tensor-map encoder cannot be had is not supported
    CUtensorMap probe;
    if (tmap_encode_bf16(&probe, weights->w_lm, cfg->hidden, cfg->vocab, (unsigned long long)cfg->hidden * 2, 64, 128) == cudaErrorNotSupported) {
      delete h;
      return DART_ERR_UNSUPPORTED_ARCH;
    }
  }
  PlanSet ps;
  build_plans(*cfg, weights, n_sm, ps);
  PlanHost* plans[5] = {&ps.fc, &ps.qkv, &ps.o, &ps.gu, &ps.down};
  {
    INIT_CHECK(tmap_encode_bf16(&h->map_lm, weights->w_lm, cfg->hidden, cfg->vocab, (unsigned long long)cfg->hidden * 2, 64, 128));
    INIT_CHECK(tmap_encode_bf16(&h->map_lm256, weights->w_lm, cfg->hidden, cfg->vocab, (unsigned long long)cfg->hidden * 2, 64, 256));
    if (cfg->feat_in > 0) {
      const unsigned long long hh = cfg->hidden, kvr = (unsigned long long)cfg->n_kv_heads * cfg->head_dim;
      const bf16* wk = static_cast<const bf16*>(weights->w_k);
      const bf16* wv = static_cast<const bf16*>(weights->w_v);
      INIT_CHECK(tmap_encode_bf16(&h->pmap_fc, weights->w_fc, cfg->feat_in, hh, (unsigned long long)cfg->feat_in * 2, 64, 256));
      INIT_CHECK(tmap_encode_bf16(&h->pmap_kv[0], wk, hh, kvr, hh * 4, 64, 256));
      INIT_CHECK(tmap_encode_bf16(&h->pmap_kv[1], wk + hh, hh, kvr, hh * 4, 64, 256));
      INIT_CHECK(tmap_encode_bf16(&h->pmap_kv[2], wv, hh, kvr, hh * 4, 64, 256));
      INIT_CHECK(tmap_encode_bf16(&h->pmap_kv[3], wv + hh, hh, kvr, hh * 4, 64, 256));
    }
    UmmaMaps* maps[5] = {&h->maps_fc, &h->maps_qkv, &h->maps_o, &h->maps_gu, &h->maps_down};
    for (int i = 0; i < 5; ++i) {
      const GemmPlan& pl = plans[i]->plan;
      for (int sg = 0; sg < pl.nseg; ++sg)
        INIT_CHECK(tmap_encode_bf16(&maps[i]->W[sg], pl.seg[sg].W, pl.Kd, pl.seg[sg].rows, (unsigned long long)pl.seg[sg].ld * 2, 64, 128));
    }
  }
  // gate / up with row ownership (umma_own.cu): weight maps with boxes of 64 k x R rows
  for (int i = 0; i < 3; ++i) {     // a plan and weight boxes of their own height per token-row padding
    h->own_ok[i] = n_sm <= 256 && own_plan_make(&h->own_gu[i], cfg->mlp_inter, cfg->hidden, n_sm, i == 0 ? 8 : (i == 1 ? 32 : 128));
    if (h->own_ok[i]) {
      const unsigned long long hh = cfg->hidden;
      INIT_CHECK(tmap_encode_bf16(&h->own_w_gu[i][0], weights->w_gate, hh, cfg->mlp_inter, hh * 2, 64, h->own_gu[i].R));
      INIT_CHECK(tmap_encode_bf16(&h->own_w_gu[i][1], weights->w_up, hh, cfg->mlp_inter, hh * 2, 64, h->own_gu[i].R));
    }
  }
  for (int i = 0; i < 5; ++i) {
    PlanHost& ph = *plans[i];
    INIT_CHECK(upload(h, ph.expected, &ph.plan.d_expected));
    INIT_CHECK(upload(h, ph.meta, &ph.plan.d_meta));
    std::vector<int> zeros(ph.plan.n_groups, 0);
    INIT_CHECK(upload(h, zeros, &ph.plan.d_ctr));
  }
  h->plan_fc = ps.fc.plan; h->plan_qkv = ps.qkv.plan; h->plan_o = ps.o.plan; h->plan_gu = ps.gu.plan; h->plan_down = ps.down.plan;
  h->lm_grid = 2 * n_sm;
  if (h->lm_grid > cfg->vocab / 16) h->lm_grid = cfg->vocab / 16;
  h->attn_pairs_cap = attn_pairs_capacity(*cfg, n_sm);

  const size_t part_cap = part_capacity(*cfg, n_sm);
  h->ws.bytes = layout_workspace(*cfg, part_cap, h->attn_pairs_cap, 2 * n_sm, nullptr, nullptr);
  INIT_CHECK(cudaMalloc(&h->ws.base, h->ws.bytes));
  layout_workspace(*cfg, part_cap, h->attn_pairs_cap, 2 * n_sm, static_cast<char*>(h->ws.base), &h->ws);
  INIT_CHECK(cudaMemset(h->ws.base, 0, h->ws.bytes));

  // the <mask> rows' z (last row of the z buffers) and the 1/rms of their g half: constants of the model
  {
    INIT_CHECK(launch_mask_row(static_cast<const bf16*>(weights->mask_vec), static_cast<const bf16*>(weights->norm_g),
                               static_cast<const bf16*>(weights->norm_e), cfg->hidden, cfg->rms_eps, h->ws.zmask_hi,
                               h->ws.zmask_lo, h->ws.rstd_mask, h->ws.mask_res, nullptr));
  }

  INIT_CHECK(launch_rope_table(h->ws.rope_tab, cfg->max_prefix + cfg->K, cfg->head_dim, cfg->rope_theta, nullptr));
  if (cfg->head_dim == 128) {   // the attention's maps over the library's own buffers
    const unsigned long long q_rows = (unsigned long long)cfg->max_batch * cfg->n_q_heads * cfg->K;
    const unsigned long long n_rows16 = (unsigned long long)cfg->max_batch * cfg->n_kv_heads * 16;
    INIT_CHECK(tmap_encode_bf16(&h->attn_maps.mapQhi, h->ws.q_hi, 128, q_rows, 256, 64, 16));
    INIT_CHECK(tmap_encode_bf16(&h->attn_maps.mapQlo, h->ws.q_lo, 128, q_rows, 256, 64, 16));
    INIT_CHECK(tmap_encode_bf16(&h->attn_maps.mapKn, h->ws.k_new, 128, n_rows16, 256, 64, 64));
    INIT_CHECK(tmap_encode_bf16(&h->attn_maps.mapVn, h->ws.v_new, 128, n_rows16, 256, 64, 64));
  }

  // Appendix D's per-level weights: fp64 from the fp32 settings, rounded once to fp32
  for (int i = 0; i < 8; ++i) {
    h->wl[i] = (float)pow((double)cfg->logit_decay, (double)i);
    h->wv[i] = (float)pow((double)(i + 1), -(double)cfg->level_exp);
  }
  h->wn = cfg->w_ng;
  h->miss = (float)log((double)cfg->eps_ng);

  // N-gram rows -> device table in the configured layout (of duplicate rows the first wins)
  const long long n_rows = ngram ? ngram->n_rows : 0;
  if (n_rows > 0) {
    if (n_rows >= (1ll << 32) - 1) { dart_draft_destroy(h); return DART_ERR_INVALID_ARG; }
    for (long long i = 0; i < n_rows; ++i) {
      const int ord = ngram->order[i];
      const int c0 = ngram->ctx0[i], c1 = ngram->ctx1[i], nx = ngram->next[i];
      if ((ord != 2 && ord != 3) || c1 < 0 || nx < 0 || c1 >= cfg->vocab || nx >= cfg->vocab ||
          (ord == 3 && (c0 < 0 || c0 >= cfg->vocab))) {
        dart_draft_destroy(h);
        return DART_ERR_INVALID_ARG;
      }
    }
  }
  if (n_rows > 0 && cfg->ngram_layout == DART_NGRAM_TRIE) {
    INIT_CHECK(ngram_trie_build(ngram->order, ngram->ctx0, ngram->ctx1, ngram->next, ngram->score, n_rows, cfg->vocab,
                                cfg->ngram_order, &h->ng_trie));
    h->ng_bytes = h->ng_trie.bytes;
  } else if (n_rows > 0) {
    // open addressing over buckets of eight rows (NgramTable in kernels.h), linear probing over buckets, load <= 0.5
    size_t cap = 16;
    while (cap < (size_t)(2 * n_rows)) cap <<= 1;
    if (cap > (1ull << 31)) { dart_draft_destroy(h); return DART_ERR_INVALID_ARG; }
    const size_t n_buckets = cap / 8;
    std::vector<NgramSlot> tab(cap);
    std::vector<uint16_t> fps(cap, 0);
    memset(tab.data(), 0, cap * sizeof(NgramSlot));
    const uint32_t mask = (uint32_t)(n_buckets - 1);
    uint32_t max_probe = 0;
    for (long long i = 0; i < n_rows; ++i) {
      const int ord = ngram->order[i];
      const int c0 = ngram->ctx0[i], c1 = ngram->ctx1[i], nx = ngram->next[i];
      if (ord == 3 && cfg->ngram_order < 3) continue;
      const unsigned long long key = ngram_key(ord, c0, c1, nx), hh = ngram_hash(key);
      const uint16_t f = (uint16_t)ngram_fingerprint(hh);
      uint32_t pos = (uint32_t)hh & mask, d = 0;
      for (;; pos = (pos + 1) & mask, ++d) {
        int slot = -1;
        bool dup = false;
        for (int q = 0; q < 8 && slot < 0 && !dup; ++q) {
          if (fps[(size_t)pos * 8 + q] == 0) slot = q;                       // slots of a bucket fill in order: none is used after an empty one
          else if (tab[(size_t)pos * 8 + q].key == key) dup = true;          // of duplicate rows the first wins
        }
        if (dup) break;
        if (slot >= 0) {
          tab[(size_t)pos * 8 + slot].key = key;
          tab[(size_t)pos * 8 + slot].score = ngram->score[i];
          fps[(size_t)pos * 8 + slot] = f;
          if (d > max_probe) max_probe = d;
          break;
        }
      }
    }
    // one allocation: the fingerprint words first (16 bytes per bucket), then the slots
    const size_t fp_bytes = align_up(n_buckets * 16, 256);
    INIT_CHECK(cudaMalloc(&h->ng_base, fp_bytes + cap * sizeof(NgramSlot)));
    INIT_CHECK(cudaMemcpy(h->ng_base, fps.data(), n_buckets * 16, cudaMemcpyHostToDevice));
    INIT_CHECK(cudaMemcpy(static_cast<char*>(h->ng_base) + fp_bytes, tab.data(), cap * sizeof(NgramSlot), cudaMemcpyHostToDevice));
    h->ng_slots = reinterpret_cast<NgramSlot*>(static_cast<char*>(h->ng_base) + fp_bytes);
    h->ng_mask = mask;
    h->ng_max_probe = max_probe;
    h->ng_bytes = fp_bytes + cap * sizeof(NgramSlot);
  }

  INIT_CHECK(topk_merge_setup(2 * n_sm));
  INIT_CHECK(attention_setup());
  INIT_CHECK(tree_setup(cfg->topk, cfg->beam, cfg->tree_budget, cfg->K));
  INIT_CHECK(cudaDeviceSynchronize());
#undef INIT_CHECK
  *out = h;
  return DART_OK;
}

int dart_draft_destroy(dart_handle* h) {
  if (h == nullptr) return DART_OK;
  for (void* p : h->owned) cudaFree(p);
  if (h->ws.base) cudaFree(h->ws.base);
  if (h->ng_base) cudaFree(h->ng_base);
  ngram_trie_free(&h->ng_trie);
  delete h;
  return DART_OK;
}

int dart_step_launch_count(const dart_handle* h, int batch, int n_fresh) {
  (void)batch;
  if (h == nullptr) return 0;
  // fc, qkv, attention, combine, o_proj, gate/up, down, lm head, merge (+ bigram sweep, tree)
  return (n_fresh > 0 ? 11 : 10);
}

int dart_draft_step(dart_handle* h, const dart_step_in* in, const dart_step_out* out, void* cuda_stream) {
  if (h == nullptr || in == nullptr || out == nullptr) return DART_ERR_INVALID_ARG;
  const dart_config& c = h->cfg;
  const int B = in->batch, K = c.K;
  if (B < 1) return DART_ERR_INVALID_ARG;
  if (B > c.max_batch) return DART_ERR_CAPACITY;
  // fresh rows per sequence: one count for all, or the caller's per-sequence counts
  FreshOffsets fo;
  fo.v[0] = 0;
  for (int b = 0; b < B; ++b) {
    const int Fb = in->fresh_counts_host != nullptr ? in->fresh_counts_host[b] : in->n_fresh;
    if (Fb < 0 || Fb > K) return DART_ERR_INVALID_ARG;
    fo.v[b + 1] = fo.v[b] + Fb;
  }
  for (int b = B + 1; b < 33; ++b) fo.v[b] = fo.v[B];
  const int NF = fo.v[B];   // fresh rows of the whole batch
  if (in->seq_lens == nullptr || in->seq_lens_host == nullptr || !aligned16(in->k_cache) || !aligned16(in->v_cache))
    return DART_ERR_INVALID_ARG;
  if (NF > 0 && (!aligned32(in->feats) || in->tokens == nullptr)) return DART_ERR_INVALID_ARG;
  if (out->topk_ids == nullptr || out->topk_slogit == nullptr) return DART_ERR_INVALID_ARG;
  long long total_keys = 0;
  for (int b = 0; b < B; ++b) {
    const int P = in->seq_lens_host[b];
    if (P < 0) return DART_ERR_INVALID_ARG;
    if ((long long)P + (fo.v[b + 1] - fo.v[b]) > c.max_prefix) return DART_ERR_CAPACITY;
    total_keys += P;
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int M = B * K, MP = padded_tokens(M);
  const int hdim = c.hidden, dq = c.n_q_heads * c.head_dim;
  Workspace& ws = h->ws;
  cudaError_t e;
  auto mark = [&](int stage, bool begin) {
    if (h->prof_stage == stage) cudaEventRecord(begin ? h->prof_start : h->prof_stop, st);
  };
  EpiArgs ep;
  GemmInput gi;
  if (h->maps_M != M) {
    // activation tensor maps: hi and lo buffers as one [M rows][2][width] tensor, box = 64 k x 2 x MP rows; rows past M
    // read as zeros
    struct { UmmaMaps* m; const bf16* hi; const bf16* lo; int width; } xin[4] = {
        {&h->maps_qkv, ws.z_hi, ws.z_lo, 2 * hdim}, {&h->maps_o, ws.a_hi, ws.a_lo, dq},
        {&h->maps_gu, ws.n_hi, ws.n_lo, hdim}, {&h->maps_down, ws.u_hi, ws.u_lo, c.mlp_inter}};
    for (int i = 0; i < 4; ++i) {
      const unsigned long long pair = (unsigned long long)(reinterpret_cast<const char*>(xin[i].lo) - reinterpret_cast<const char*>(xin[i].hi));
      if ((e = tmap_encode_bf16_pair(&xin[i].m->Xhi, xin[i].hi, pair, xin[i].width, M, (unsigned long long)xin[i].width * 2, MP)) != cudaSuccess)
        return fail_cuda(h, e);
    }
    h->maps_M = M;
  }
  auto project = [&](const GemmPlan& plan, const UmmaMaps& maps) -> cudaError_t {
    return launch_umma_rows(plan, maps, gi, ep, ws.part, ws.status, st);
  };
  const int own_i = MP == 8 ? 0 : (MP == 32 ? 1 : 2);
  const bool own_gu = h->own_ok[own_i];      // gate / up with row ownership: no pieces, no finalize

  // the <mask> rows of z are constant; they are (re)written only when the row pattern changes
  if (h->z_B != B || memcmp(h->z_foff.v, fo.v, sizeof(fo.v)) != 0) {
    if ((e = launch_fill_mask_rows(ws.z_hi, ws.z_lo, ws.zmask_hi, ws.zmask_lo, B, K, fo, 2 * hdim, st)) != cudaSuccess) return fail_cuda(h, e);
    h->z_B = B; h->z_foff = fo;
  }
  auto set_epi = [&](int mode) {
    memset(&ep, 0, sizeof(ep));
    ep.mode = mode; ep.K = K; ep.h = hdim; ep.eps = c.rms_eps; ep.B = B; ep.status = ws.status;
    memcpy(ep.foff, fo.v, sizeof(ep.foff));
  };

  // S0: feature-fusion FC on the fresh rows; epilogue: residual g, z g-half (gain-scaled), sums of squares;
  // prologue: z e-half = RMSNorm(embedding of the next token)
  mark(0, true);
  if (NF > 0) {
    set_epi(EPI_FC);
    ep.res0 = ws.res0; ep.gamma = static_cast<const bf16*>(h->w.norm_g);
    ep.out_hi = ws.z_hi; ep.out_lo = ws.z_lo; ep.ld_out = 2 * hdim; ep.ss_out = ws.ss_g;
    ep.tokens = in->tokens; ep.vocab = c.vocab; ep.embed = static_cast<const bf16*>(h->w.embed);
    ep.gamma_e = static_cast<const bf16*>(h->w.norm_e);
    if (c.feat_in == 0) {   // the caller fused the features: feats = g [fresh rows][hidden]
      if ((e = launch_prefused_rows(ep, static_cast<const bf16*>(in->feats), NF, st)) != cudaSuccess) return fail_cuda(h, e);
    } else {
    gi = {static_cast<const bf16*>(in->feats), nullptr, c.feat_in, NF};
    if ((h->maps_feats != in->feats || h->maps_fc_M != NF)) {
      // plain bf16 input: one box of 2 * MP rows, the rows past the fresh rows (the "lo" half among them) read as zeros
      if ((e = tmap_encode_bf16(&h->maps_fc.Xhi, in->feats, c.feat_in, NF, (unsigned long long)c.feat_in * 2, 64,
                                2 * padded_tokens(NF))) != cudaSuccess)
        return fail_cuda(h, e);
      h->maps_feats = in->feats; h->maps_fc_M = NF;
    }
    if ((e = project(h->plan_fc, h->maps_fc)) != cudaSuccess) return fail_cuda(h, e);
    }
  }
  mark(0, false);

  // S1: QKV projection; epilogue: 1/rms of g, RoPE, q and new k/v as hi/lo, cache append
  mark(1, true);
  set_epi(EPI_QKV);
  ep.ss_in = ws.ss_g; ep.ss_tiles = h->h_tiles; ep.ss_mp = padded_tokens(NF > 0 ? NF : 1); ep.rstd_mask = ws.rstd_mask;
  ep.Hq = c.n_q_heads; ep.Hkv = c.n_kv_heads; ep.dh = c.head_dim; ep.seq_lens = in->seq_lens; ep.rope_tab = ws.rope_tab;
  ep.q_hi = ws.q_hi; ep.q_lo = ws.q_lo; ep.k_new = ws.k_new; ep.v_new = ws.v_new;
  ep.k_cache = static_cast<bf16*>(in->k_cache); ep.v_cache = static_cast<bf16*>(in->v_cache); ep.P_cap = c.max_prefix;
  gi = {ws.z_hi, ws.z_lo, 2 * hdim, M};
  if ((e = project(h->plan_qkv, h->maps_qkv)) != cudaSuccess) return fail_cuda(h, e);
  mark(1, false);

  // S2: split-KV attention over cache rows 0 .. P_b-1 and the K new rows
  mark(2, true);
  AttnParams ap;
  ap.B = B; ap.K = K; ap.Hq = c.n_q_heads; ap.Hkv = c.n_kv_heads; ap.dh = c.head_dim;
  ap.seq_lens = in->seq_lens; ap.q_hi = ws.q_hi; ap.q_lo = ws.q_lo; ap.k_new = ws.k_new; ap.v_new = ws.v_new;
  ap.k_cache = static_cast<const bf16*>(in->k_cache); ap.v_cache = static_cast<const bf16*>(in->v_cache); ap.P_cap = c.max_prefix;
  ap.o_part = ws.o_part; ap.ml_part = ws.ml_part; ap.a_hi = ws.a_hi; ap.a_lo = ws.a_lo;
  const AttnUmmaMaps* amaps = nullptr;
  if (c.head_dim == 128 && (long long)c.max_batch * c.n_kv_heads * c.max_prefix < (1ll << 31)) {
    // maps over the caller's caches are re-encoded only when the pointers change
    if (h->attn_k_ptr != in->k_cache || h->attn_v_ptr != in->v_cache) {
      const unsigned long long rows = (unsigned long long)c.max_batch * c.n_kv_heads * c.max_prefix;
      if ((e = tmap_encode_bf16(&h->attn_maps.mapK, in->k_cache, 128, rows, 256, 64, 64)) != cudaSuccess ||
          (e = tmap_encode_bf16(&h->attn_maps.mapV, in->v_cache, 128, rows, 256, 64, 64)) != cudaSuccess)
        return fail_cuda(h, e);
      h->attn_k_ptr = in->k_cache; h->attn_v_ptr = in->v_cache;
    }
    amaps = &h->attn_maps;
  }
  {
    // one chunk per CTA, about two CTAs per SM, 128 .. 512 keys; the tcgen05 split has its own rule
    long long per = (total_keys * c.n_kv_heads + 2 * h->n_sm - 1) / (2 * h->n_sm);
    long long chunk = ((per + 63) / 64) * 64;
    if (chunk < 128) chunk = 128;
    if (chunk > kAttnMaxChunk) chunk = kAttnMaxChunk;
    if (attn_uses_umma(B, c.n_kv_heads, c.head_dim, in->seq_lens_host, amaps != nullptr)) {
      const int uc = attn_umma_chunk_keys(B, c.n_kv_heads, in->seq_lens_host, h->n_sm, h->attn_pairs_cap);
      if (uc > 0) chunk = uc;
    }
    ap.chunk_keys = (int)chunk;
    long long pairs = 0;
    for (int b = 0; b < B; ++b) pairs += (in->seq_lens_host[b] + ap.chunk_keys - 1) / ap.chunk_keys + 1;
    if (pairs > h->attn_pairs_cap) return DART_ERR_INTERNAL;
  }
  if ((e = launch_attention(ap, in->seq_lens_host, amaps, ws.status, st)) != cudaSuccess) return fail_cuda(h, e);
  mark(2, false);

  // S3: o_proj; epilogue: x1 = residual + proj, gain-scaled hi/lo, sums of squares
  mark(3, true);
  set_epi(EPI_RES);
  ep.res0 = ws.res0; ep.res_in = nullptr; ep.res_out = ws.x1; ep.mask_res = ws.mask_res;
  ep.gamma = static_cast<const bf16*>(h->w.norm_post);
  ep.out_hi = ws.n_hi; ep.out_lo = ws.n_lo; ep.ld_out = hdim; ep.ss_out = ws.ss_1;
  gi = {ws.a_hi, ws.a_lo, dq, M};
  if ((e = project(h->plan_o, h->maps_o)) != cudaSuccess) return fail_cuda(h, e);
  mark(3, false);

  // S4: gate/up; epilogue: u = SiLU(rstd1 * gate) * (rstd1 * up)
  mark(4, true);
  set_epi(EPI_GATE_UP);
  ep.ss_in = ws.ss_1; ep.ss_tiles = h->h_tiles; ep.ss_mp = MP;
  ep.out_hi = ws.u_hi; ep.out_lo = ws.u_lo; ep.ld_out = c.mlp_inter;
  gi = {ws.n_hi, ws.n_lo, hdim, M};
  if (own_gu) e = launch_umma_own(h->own_gu[own_i], h->own_w_gu[own_i], h->maps_gu.Xhi, M, ep, ws.status, st);
  else e = project(h->plan_gu, h->maps_gu);
  if (e != cudaSuccess) return fail_cuda(h, e);
  mark(4, false);

  // S5: down; epilogue: x2 = x1 + proj, gain-scaled hi/lo for the LM head, sums of squares
  mark(5, true);
  set_epi(EPI_RES);
  ep.res_in = ws.x1; ep.res_out = nullptr; ep.gamma = static_cast<const bf16*>(h->w.norm_final);
  ep.out_hi = ws.n_hi; ep.out_lo = ws.n_lo; ep.ld_out = hdim; ep.ss_out = ws.ss_2;
  gi = {ws.u_hi, ws.u_lo, c.mlp_inter, M};
  if ((e = project(h->plan_down, h->maps_down)) != cudaSuccess) return fail_cuda(h, e);
  mark(5, false);

  // S6 + S7: LM head with fused log-softmax / top-k, then the merge
  LmParams lp;
  lp.W = static_cast<const bf16*>(h->w.w_lm); lp.V = c.vocab; lp.Kd = hdim;
  lp.x_hi = ws.n_hi; lp.x_lo = ws.n_lo; lp.ldx = hdim; lp.M = M; lp.K = K;
  lp.ss_in = ws.ss_2; lp.ss_tiles = h->h_tiles; lp.ss_mp = MP; lp.rms_eps = c.rms_eps;
  lp.topk = c.topk;
  lp.inv_temp = c.temperature > 0.f ? 1.f / c.temperature : 1.f;
  lp.gumbel = c.temperature > 0.f ? 1 : 0;
  lp.seed_lo = (uint32_t)(c.philox_seed & 0xffffffffull); lp.seed_hi = (uint32_t)(c.philox_seed >> 32);
  lp.step = (uint32_t)(in->step_counter & 0xffffffffull);
  lp.eps_logit = c.eps_logit;
  lp.grid = (MP <= 32) ? h->lm_grid : (h->lm_grid + 1) / 2;
  lp.logits_out = out->logits;
  lp.part_stats = ws.lm_stats; lp.part_key = ws.lm_key; lp.part_y = ws.lm_y; lp.part_id = ws.lm_id;
  lp.out_ids = out->topk_ids; lp.out_slogit = out->topk_slogit;
  mark(6, true);
  {
    // one CTA per SM at most: the CTAs of this kernel wait on one another's pieces, so all must be resident
    const bool dense = MP == 128;   // many token rows: tokens on the MMA's M side, 256 vocabulary rows per tile
    const long long units = lm_head_units(c.vocab, hdim, dense);
    lp.grid = (int)(units < h->n_sm ? units : h->n_sm);
    if (dense) {
      if (h->lmx_M != M) {
        if ((e = tmap_encode_bf16(&h->lmx_hi, ws.n_hi, hdim, M, (unsigned long long)hdim * 2, 64, 128)) != cudaSuccess ||
            (e = tmap_encode_bf16(&h->lmx_lo, ws.n_lo, hdim, M, (unsigned long long)hdim * 2, 64, 128)) != cudaSuccess)
          return fail_cuda(h, e);
        h->lmx_M = M;
      }
      e = launch_lm_head_dense(lp, h->map_lm256, h->lmx_hi, h->lmx_lo, ws.lm_pieces, ws.lm_flags, ++h->lm_tag, ws.status, ws.lm_bound, st);
    } else {
      e = launch_lm_head_umma(lp, h->map_lm, h->maps_gu.Xhi, ws.lm_pieces, ws.lm_flags, ++h->lm_tag, ws.status, st);
    }
  }
  if (e != cudaSuccess) return fail_cuda(h, e);
  mark(6, false);
  mark(7, true);
  if ((e = launch_topk_merge(lp, st)) != cudaSuccess) return fail_cuda(h, e);
  mark(7, false);
  if (h->prof_stage >= 0 && h->prof_stage <= 7) h->prof_stage = -1;
  return DART_OK;
}

int dart_tree_verify_inputs(dart_handle* h, const dart_verify_in* in, const dart_verify_out* out, void* cuda_stream) {
  if (h == nullptr || in == nullptr || out == nullptr) return DART_ERR_INVALID_ARG;
  const dart_config& c = h->cfg;
  if (in->batch < 1 || in->max_levels < 1 || in->max_levels > 64 || c.tree_budget > 64) return DART_ERR_INVALID_ARG;
  if (in->batch > c.max_batch) return DART_ERR_CAPACITY;
  if (in->parents == nullptr || in->depth == nullptr || in->n_nodes == nullptr || in->root_pos == nullptr ||
      out->position_ids == nullptr || out->retrieve == nullptr || out->n_leaves == nullptr)
    return DART_ERR_INVALID_ARG;
  const cudaError_t e = launch_verify_inputs(in->batch, c.tree_budget, in->max_levels, in->parents, in->depth, in->n_nodes, in->root_pos,
                                             out->position_ids, out->retrieve, out->n_leaves, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? DART_OK : fail_cuda(h, e);
}

namespace {
bool train_attn_dims_ok(int batch, int n_kv_heads, int head_dim, int prompt_len, int draft_len) {
  return batch >= 1 && batch <= 64 && n_kv_heads >= 1 && head_dim == 128 && prompt_len >= 1 && draft_len >= 1 && draft_len <= 16 &&
         (long long)batch * n_kv_heads * prompt_len * (1 + draft_len) < (1ll << 31) / 128;
}
}  // namespace

int dart_train_attention_fwd(const dart_train_attn_in* in, void* cuda_stream) {
  if (in == nullptr) return DART_ERR_INVALID_ARG;
  if (!train_attn_dims_ok(in->batch, in->n_kv_heads, in->head_dim, in->prompt_len, in->draft_len)) return DART_ERR_INVALID_ARG;
  if (in->n_q_heads < 1 || in->n_q_heads % in->n_kv_heads != 0 || in->n_q_heads > 65535) return DART_ERR_INVALID_ARG;
  if (!aligned16(in->q) || !aligned16(in->k) || !aligned16(in->v) || !aligned16(in->out) || in->seq_lens_host == nullptr)
    return DART_ERR_INVALID_ARG;
  for (int b = 0; b < in->batch; ++b)
    if (in->seq_lens_host[b] < 0 || in->seq_lens_host[b] > in->prompt_len) return DART_ERR_INVALID_ARG;
  int dev = 0, major = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail_cuda(nullptr, e);
  e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  if (e != cudaSuccess) return fail_cuda(nullptr, e);
  if (major != 10) return DART_ERR_UNSUPPORTED_ARCH;

  const int B = in->batch, Hq = in->n_q_heads, Hkv = in->n_kv_heads, Lp = in->prompt_len, d = in->draft_len;
  const unsigned long long L = (unsigned long long)Lp * (1 + d);
  TrainAttnArgs a;
  memset(&a, 0, sizeof(a));
  if ((e = tmap_encode_bf16(&a.mapQ, in->q, 128, (unsigned long long)B * Hq * L, 256, 64, 128)) != cudaSuccess ||
      (e = tmap_encode_bf16(&a.mapK, in->k, 128, (unsigned long long)B * Hkv * L, 256, 64, 128)) != cudaSuccess ||
      (e = tmap_encode_bf16(&a.mapV, in->v, 128, (unsigned long long)B * Hkv * L, 256, 64, 64)) != cudaSuccess)
    return e == cudaErrorNotSupported ? DART_ERR_UNSUPPORTED_ARCH : fail_cuda(nullptr, e);
  a.B = B; a.Hq = Hq; a.Hkv = Hkv; a.prompt_len = Lp; a.draft_len = d; a.n_clean_tiles = (Lp + 127) / 128;
  for (int b = 0; b < B; ++b) a.seq_len[b] = in->seq_lens_host[b];
  a.scale_log2e = (float)(1.4426950408889634 / sqrt(128.0));
  a.out = static_cast<bf16*>(in->out);
  a.status = in->status;
  e = launch_train_attn(a, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? DART_OK : fail_cuda(nullptr, e);
}

int dart_draft_prefill(dart_handle* h, const dart_prefill_in* in, void* cuda_stream) {
  if (h == nullptr || in == nullptr) return DART_ERR_INVALID_ARG;
  const dart_config& c = h->cfg;
  const int B = in->batch, K = c.K, hdim = c.hidden;
  if (B < 1) return DART_ERR_INVALID_ARG;
  if (B > c.max_batch) return DART_ERR_CAPACITY;
  if (in->seq_lens_host == nullptr || in->new_rows_host == nullptr || !aligned16(in->k_cache) || !aligned16(in->v_cache))
    return DART_ERR_INVALID_ARG;
  if (c.feat_in <= 0) return DART_ERR_INVALID_ARG;
  long long total = 0;
  for (int b = 0; b < B; ++b) {
    const int P = in->seq_lens_host[b], N = in->new_rows_host[b];
    if (P < 0 || N < 0) return DART_ERR_INVALID_ARG;
    if ((long long)P + N > c.max_prefix) return DART_ERR_CAPACITY;
    total += N;
  }
  if (total == 0) return DART_OK;
  if (!aligned32(in->feats) || in->tokens == nullptr) return DART_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  Workspace& ws = h->ws;
  const bf16* feats = static_cast<const bf16*>(in->feats);
  cudaError_t e;
  // passes of up to kPrefillPassRows packed rows: feature FC -> z g-half, beside it embeddings -> z e-half, then k / v -> caches
  for (long long done = 0; done < total; done += kPrefillPassRows) {
    const int T = (int)(total - done < kPrefillPassRows ? total - done : kPrefillPassRows);
    DenseArgs a;
    memset(&a, 0, sizeof(a));
    a.T = T; a.h = hdim; a.eps = c.rms_eps; a.status = ws.status;
    a.z = ws.pz; a.ldz = 2 * hdim; a.ss = ws.pss; a.ss_ld = prefill_fc_tiles(c); a.ss_n = prefill_fc_tiles(c);
    // where the pass's rows go: sequence b contributes rows [lo, hi) of its new rows
    a.B = B;
    long long off = 0;
    for (int b = 0; b < B; ++b) {
      const long long lo = done > off ? done - off : 0;                       // first of b's new rows in this pass
      long long hi = done + T - off;                                           // one past the last
      if (hi > in->new_rows_host[b]) hi = in->new_rows_host[b];
      if (hi < lo) hi = lo;
      a.seq_off[b] = (int)(off + lo - done < 0 ? 0 : off + lo - done);
      a.seq_P[b] = in->seq_lens_host[b] + (int)lo;
      off += in->new_rows_host[b];
      a.seq_off[b + 1] = (int)(a.seq_off[b] + (hi - lo));
    }
    for (int b = B + 1; b < 33; ++b) a.seq_off[b] = a.seq_off[B];
    DenseArgs fc = a;
    fc.mode = 0; fc.n_w = 1; fc.n_tiles_per_w = prefill_fc_tiles(c); fc.n_out = hdim;
    fc.KB[0] = (c.feat_in + 63) / 64; fc.KB[1] = 0; fc.a_koff[0] = 0; fc.a_koff[1] = 0;
    fc.gain = static_cast<const bf16*>(h->w.norm_g);
    fc.mapW[0] = h->pmap_fc;
    if ((e = tmap_encode_bf16(&fc.mapA, feats + (size_t)done * c.feat_in, c.feat_in, T, (unsigned long long)c.feat_in * 2, 64, 128)) != cudaSuccess)
      return fail_cuda(h, e);
    if ((e = launch_umma_dense(fc, h->n_sm, st)) != cudaSuccess) return fail_cuda(h, e);
    if ((e = launch_prefill_embed(in->tokens + done, T, c.vocab, static_cast<const bf16*>(h->w.embed),
                                  static_cast<const bf16*>(h->w.norm_e), hdim, c.rms_eps, ws.pz, 2 * hdim, h->n_sm, st)) != cudaSuccess)
      return fail_cuda(h, e);
    DenseArgs kv = a;
    kv.mode = 1; kv.n_w = 2; kv.n_tiles_per_w = (c.n_kv_heads * c.head_dim + 255) / 256; kv.n_out = c.n_kv_heads * c.head_dim;
    kv.KB[0] = kv.KB[1] = (hdim + 63) / 64; kv.a_koff[0] = 0; kv.a_koff[1] = hdim;
    kv.Hkv = c.n_kv_heads; kv.dh = c.head_dim; kv.rope_tab = ws.rope_tab;
    kv.k_cache = static_cast<bf16*>(in->k_cache); kv.v_cache = static_cast<bf16*>(in->v_cache); kv.P_cap = c.max_prefix;
    for (int i = 0; i < 4; ++i) kv.mapW[i] = h->pmap_kv[i];
    if ((e = tmap_encode_bf16(&kv.mapA, ws.pz, 2 * hdim, T, (unsigned long long)hdim * 4, 64, 128)) != cudaSuccess) return fail_cuda(h, e);
    if ((e = launch_umma_dense(kv, h->n_sm, st)) != cudaSuccess) return fail_cuda(h, e);
  }
  return DART_OK;
}

int dart_build_tree(dart_handle* h, const dart_tree_in* in, const dart_tree_out* out, void* cuda_stream) {
  if (h == nullptr || in == nullptr || out == nullptr) return DART_ERR_INVALID_ARG;
  const dart_config& c = h->cfg;
  if (in->batch < 1 || in->first_row < 0 || in->n_levels < 1 || in->first_row + in->n_levels > c.K) return DART_ERR_INVALID_ARG;
  if (in->batch > c.max_batch) return DART_ERR_CAPACITY;
  if (in->topk_ids == nullptr || in->topk_slogit == nullptr || in->ctx_tail == nullptr) return DART_ERR_INVALID_ARG;
  if (out->tokens == nullptr || out->parents == nullptr || out->depth == nullptr || out->mask == nullptr || out->n_nodes == nullptr)
    return DART_ERR_INVALID_ARG;
  if (in->n_levels * (c.tree_budget - 1) > 1024) return DART_ERR_INVALID_ARG;
  TreeParams tp;
  tp.B = in->batch; tp.K = c.K; tp.topk = c.topk; tp.beam = c.beam; tp.budget = c.tree_budget;
  tp.first_row = in->first_row; tp.n_levels = in->n_levels; tp.ngram_order = c.ngram_order; tp.vocab = c.vocab;
  for (int b = 0; b < 32; ++b) {  // per-sequence first logit row (level 0); a sequence has min(n_levels, K - first row) levels
    int fr = in->first_row;
    if (in->first_rows_host != nullptr && b < in->batch) {
      fr = in->first_rows_host[b];
      if (fr < 0 || fr >= c.K) return DART_ERR_INVALID_ARG;
    }
    tp.first_rows[b] = (unsigned char)fr;
  }
  tp.ids = in->topk_ids; tp.slogit = in->topk_slogit; tp.ctx_tail = in->ctx_tail;
  tp.table.fp = static_cast<const uint4*>(h->ng_base); tp.table.slots = h->ng_slots; tp.table.mask = h->ng_mask; tp.table.max_probe = h->ng_max_probe;
  for (int i = 0; i < 8; ++i) { tp.wl[i] = h->wl[i]; tp.wv[i] = h->wv[i]; }
  tp.trie.bi_off = h->ng_trie.bi_off; tp.trie.bi_ent = h->ng_trie.bi_ent; tp.trie.tri_off = h->ng_trie.tri_off;
  tp.trie.tri_node = h->ng_trie.tri_node; tp.trie.tri_ent = h->ng_trie.tri_ent; tp.trie.nb8 = 8u * (uint32_t)((c.vocab + 479) / 480);
  tp.wn = h->wn; tp.miss = h->miss; tp.sg = h->ws.sg; tp.bg = h->ws.bg; tp.cx = h->ws.cx;
  tp.tokens = out->tokens; tp.parents = out->parents; tp.depth = out->depth; tp.mask = out->mask;
  tp.n_nodes = out->n_nodes; tp.scores = out->scores; tp.status = h->ws.status;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (h->prof_stage == 8) cudaEventRecord(h->prof_start, st);
  cudaError_t e = launch_tree(tp, st);
  if (e != cudaSuccess) return fail_cuda(h, e);
  if (h->prof_stage == 8) { cudaEventRecord(h->prof_stop, st); h->prof_stage = -1; }
  return DART_OK;
}

int dart_draft_step_host(dart_handle* h, const dart_host_io* io, const dart_step_in* in, const dart_step_out* out,
                         const dart_tree_in* tree_in, const dart_tree_out* tree_out, void* cuda_stream) {
  if (h == nullptr || io == nullptr) return DART_ERR_INVALID_ARG;
  if ((io->in_bytes > 0 && (io->in_host == nullptr || io->in_dev == nullptr)) ||
      (io->out_bytes > 0 && (io->out_host == nullptr || io->out_dev == nullptr)))
    return DART_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e;
  if (io->in_bytes > 0 && (e = cudaMemcpyAsync(io->in_dev, io->in_host, io->in_bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess)
    return fail_cuda(h, e);
  int rc = dart_draft_step(h, in, out, cuda_stream);
  if (rc == DART_OK) rc = dart_build_tree(h, tree_in, tree_out, cuda_stream);
  if (rc == DART_OK && io->out_bytes > 0 &&
      (e = cudaMemcpyAsync(io->out_host, io->out_dev, io->out_bytes, cudaMemcpyDeviceToHost, st)) != cudaSuccess)
    rc = fail_cuda(h, e);
  // whatever was enqueued is waited for, also after an error: the caller's buffers are quiet on return
  if ((e = cudaStreamSynchronize(st)) != cudaSuccess && rc == DART_OK) rc = fail_cuda(h, e);
  return rc;
}

int dart_set_profile_events(dart_handle* h, int stage, void* start_event, void* stop_event) {
  if (h == nullptr || stage < 0 || stage > 8 || start_event == nullptr || stop_event == nullptr) return DART_ERR_INVALID_ARG;
  h->prof_stage = stage;
  h->prof_start = static_cast<cudaEvent_t>(start_event);
  h->prof_stop = static_cast<cudaEvent_t>(stop_event);
  return DART_OK;
}

int dart_last_device_status(dart_handle* h, void* cuda_stream) {
  if (h == nullptr) return DART_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int v = 0;
  cudaError_t e = cudaMemcpyAsync(&v, h->ws.status, sizeof(int), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return fail_cuda(h, e);
  if (v != 0) {
    // A kernel gave up on a wait: the step's outputs are void, and CTAs that left between their tickets and their
    // finalize have left group counters behind.  Clear them with the status word, so that the handle's next
    // step starts from the state dart_draft_init left.
    cudaMemsetAsync(h->ws.status, 0, sizeof(int), st);
    const GemmPlan* plans[5] = {&h->plan_fc, &h->plan_qkv, &h->plan_o, &h->plan_gu, &h->plan_down};
    for (int i = 0; i < 5; ++i) cudaMemsetAsync(plans[i]->d_ctr, 0, sizeof(int) * (size_t)plans[i]->n_groups, st);
    e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return fail_cuda(h, e);
  }
  return v == 0 ? DART_OK : (v == DART_ERR_INTERNAL ? DART_ERR_INTERNAL : DART_ERR_TIMEOUT);
}

int dart_selftest_bounded_wait(dart_handle* h, int32_t spin_limit, int32_t leave_ticket, void* cuda_stream) {
  if (h == nullptr || spin_limit < 1 || spin_limit > 100000) return DART_ERR_INVALID_ARG;
  const cudaError_t e = launch_bounded_wait_probe(spin_limit, h->ws.status, leave_ticket ? h->plan_qkv.d_ctr : nullptr,
                                                  static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? DART_OK : fail_cuda(h, e);
}

}  // extern "C"
