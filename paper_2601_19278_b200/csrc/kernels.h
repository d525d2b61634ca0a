// Internal interface between the C-ABI layer (api.cu) and the kernel translation units.
#pragma once
#include <cuda_bf16.h>
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

namespace dart {

typedef __nv_bfloat16 bf16;

// Function attributes are per device: a (device, function) pair is configured the first time it is launched.
// Process-wide table behind a mutex (handles on different devices or threads may launch the same kernel).
inline bool first_launch_on_device(const void* fn, int what) {
  static std::mutex mu;
  static struct { const void* fn; int dev, what; } seen[256];
  static int n = 0;
  int dev = 0;
  cudaGetDevice(&dev);
  std::lock_guard<std::mutex> lock(mu);
  for (int i = 0; i < n; ++i)
    if (seen[i].fn == fn && seen[i].dev == dev && seen[i].what == what) return false;
  if (n < 256) { seen[n].fn = fn; seen[n].dev = dev; seen[n].what = what; ++n; }
  return true;
}

// All kernels of the step ask for the same (largest) shared-memory carve-out: the streaming kernels need
// ~200 KB per SM, and an SM whose L1 / shared-memory split differs from what the next kernel wants has to
// drain and reconfigure first, which serialises consecutive kernels and costs tens of microseconds a switch.
inline void prefer_max_shared(const void* fn) {
  if (first_launch_on_device(fn, 0))
    cudaFuncSetAttribute(fn, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
}
// Opt-in to more than 48 KB of dynamic shared memory, once per device.
inline cudaError_t allow_dynamic_smem(const void* fn, size_t bytes) {
  if (!first_launch_on_device(fn, 1)) return cudaSuccess;
  return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

// The cudaError_t behind a DART_ERR_CUDA of a call that has no handle (dart_last_cuda_error(NULL) reads it; api.cu).
void record_global_cuda_error(cudaError_t e);

// Launch with programmatic stream serialization (see pdl_wait / pdl_trigger in common.cuh).
template <class... KArgs, class... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  prefer_max_shared(reinterpret_cast<const void*>(kernel));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---------------------------------------------------------------------------------------------
// Weight-streaming small-M GEMM:  y = W[rows, Kd] * x[M, Kd]^T, split over the flattened
// (128-row tile, 64-wide k-step) space so that every CTA streams the same number of weight bytes.
// A CTA writes one fp32 partial per tile it touches; the CTA that completes a tile (or a pair of
// tiles) sums the partials in CTA order and applies the op that follows the projection.
// ---------------------------------------------------------------------------------------------
struct GemmSeg {
  const bf16* W;  // first element of the segment's sub-matrix (row 0, first column used)
  int rows;       // multiple of 16
  int tile0;      // index of this segment's first 128-row tile in the launch
  int ld;         // row stride of W in elements
  int xoff;       // column offset into the activation rows for this segment
};

constexpr int kUmmaKS = 2;         // 64-k blocks per ring stage of the stream-K projections = per work unit of their plans
constexpr int kMetaStride = 36;   // ints per 16-row tile in the piece table: count + up to 35 offsets

struct GemmPlan {
  int nseg;
  GemmSeg seg[6];
  int Kd;           // reduction length per segment, multiple of 16
  int SK;           // ceil(Kd / 64) k-blocks per row
  int KR;           // ring stages (work units) per 128-row tile = ceil(SK / kUmmaKS)
  int n_tiles;      // 128-row tiles over all segments
  int grid;         // CTAs
  int slots;        // max tiles a CTA touches
  long long U;      // n_tiles * KR work units
  int pair_offset;  // > 0: tiles T and T + pair_offset are finalized together (group = T % pair_offset)
  int n_groups;
  int* d_ctr;         // DEVICE [n_groups] tickets taken (zero between launches)
  int* d_expected;    // DEVICE [n_groups] tickets that complete a group
  int* d_meta;        // DEVICE [n_tiles*8][meta_stride]: piece count, then piece offsets (CTA order) per 16-row tile
  int meta_stride;    // <= kMetaStride
};

__host__ __device__ inline int padded_tokens(int M) { return M <= 8 ? 8 : (M <= 32 ? 32 : 128); }

struct GemmInput {
  const bf16* x_hi; const bf16* x_lo;  // [rows, ldx] activations as hi (+ lo, may be NULL)
  long long ldx;
  int M;              // valid tokens
};

enum EpiMode : int { EPI_FC = 0, EPI_QKV = 1, EPI_RES = 2, EPI_GATE_UP = 3 };

// Everything the fused epilogues need (unused fields stay zero).
struct EpiArgs {
  int mode;
  int K, h;           // rows per sequence, hidden
  // Fresh rows: sequence b's rows r < F_b carry fresh target features, F_b = foff[b+1] - foff[b]; fresh row (b, r)
  // is row foff[b] + r of the packed fresh arrays (features, tokens, g, sums of squares).  foff[B] = their count.
  int B; int foff[33];
  float eps;
  // EPI_FC: g -> res0 [B*F, h], z g-half (gain-scaled, hi/lo, row stride ld_out), ss_out [tile][MP]
  // EPI_RES: x = res + proj -> res_out, out_hi/lo = x * gamma, ss_out
  float* res0;            // FC: out; RES with res_in == NULL: the fresh rows' g
  const float* res_in;    // RES: residual in (NULL: first residual = g or <mask>)
  float* res_out;         // RES: residual out (may be NULL)
  const float* mask_res;  // g half of the <mask> representation as fp32 [h]: the <mask> rows' first residual
  const bf16* gamma;      // gain applied to the hi/lo output
  bf16* out_hi; bf16* out_lo; long long ld_out;
  float* ss_out;
  // rstd of the *input* of this projection, applied to its output: per-tile sums of squares
  const float* ss_in; int ss_tiles; int ss_mp;
  const float* rstd_mask;  // QKV: 1/rms of the <mask> row's g half
  // EPI_FC prologue: shifted token embedding of the fresh rows
  const int32_t* tokens; int vocab; const bf16* embed; const bf16* gamma_e;
  // EPI_QKV
  int Hq, Hkv, dh; const int32_t* seq_lens; const float2* rope_tab;  // [positions][dh/2] (cos, sin)
  bf16* q_hi; bf16* q_lo; bf16* k_new; bf16* v_new; bf16* k_cache; bf16* v_cache; long long P_cap;
  int* status;   // device status word (the debug build's index checks report here)
};

// The weight sub-matrices and the activations of one streaming launch.
struct StreamArgs {
  GemmSeg seg[6];     // sub-matrices streamed by this launch; tile0 in 128-row tiles
  int nseg;
  int Kd;             // reduction length (multiple of 16)
  int SK;             // 64-wide k-blocks per row
  int KR;             // ring stages (work units) per 128-row tile = ceil(SK / kUmmaKS)
  const bf16* x_hi;   // activations [rows, ldx] hi part
  const bf16* x_lo;   // lo part (== x_hi when the input is plain bf16)
  long long ldx;
  int M;              // valid token rows
};

struct GemmArgs {
  StreamArgs s;
  int slots;
  long long U;
  float* part;        // [grid][slots] pieces of 16 x MP floats
  int* ctr; const int* expected; int pair_offset;
  const int* meta; int meta_stride;
  EpiArgs epi;
};

// The projections (umma_gemm.cu): plan units are (128-row tile, 64-k block), one persistent CTA per SM.  Tensor maps: one per weight segment; Xhi = the activations: hi + lo inputs as one
// 3-D map (box = 64 k x (hi, lo) x MP rows: accumulator column 2t is token t's hi part, 2t+1 its lo part); a
// plain-bf16 input as a 2-D map with a box of 2*MP rows whose missing rows read 0 (column t is token t).
struct UmmaMaps {
  CUtensorMap W[6];
  CUtensorMap Xhi;   // the activations (see above)
};
struct UmmaGemmArgs {
  GemmArgs g;
  CUtensorMap mapW[6];
  CUtensorMap mapXhi;
  int has_lo;
  int* status;   // device status word (DEV_TIMEOUT when a bounded wait ran out)
};
cudaError_t launch_umma_rows(const GemmPlan& plan, const UmmaMaps& maps, const GemmInput& in, const EpiArgs& epi, float* part,
                             int* status, cudaStream_t st);
// Gate / up with row ownership (umma_own.cu): CTA c owns output rows [c * rows / grid, (c + 1) * rows / grid) of both
// matrices over the whole reduction length; a stage holds its rows of both for one k-block and one activation slice.
constexpr int kOwnMinRows = 96;   // rows per stage (both matrices together) from which the TMA boxes stream at the HBM rate
struct OwnPlan {
  int rows, Kd, KB;            // output rows per matrix, reduction length, 64-k blocks
  int grid, R;                 // CTAs, weight rows per TMA box = ceil(rows / grid)
  int stages, stage_bytes, w_tx_bytes;
  size_t smem;
};
struct OwnArgs {
  CUtensorMap mapW[2];         // gate and up, boxes of 64 k x R rows
  CUtensorMap mapX;            // the activations: hi + lo pair as one 3-D map
  int rows, KB, M;
  int stages, stage_bytes, w_tx_bytes;
  const float* ss_in; int ss_tiles, ss_mp, h; float eps;   // the input's sums of squares (1/rms is applied to the output)
  bf16* out_hi; bf16* out_lo; long long ld_out;
  int* status;
};
// A plan per token-row padding MP = 8, 32, 128 (the activation slice's size decides the stage count).  false: the shape
// does not suit the kernel (fewer than kOwnMinRows / 2 rows per CTA and matrix, or more than 256 -- 128 at MP = 128).
bool own_plan_make(OwnPlan* p, int rows, int Kd, int n_sm, int MP);
cudaError_t launch_umma_own(const OwnPlan& plan, const CUtensorMap* mapW, const CUtensorMap& mapX, int M, const EpiArgs& epi, int* status,
                            cudaStream_t st);

// Dense projections of the draft-side prefill (umma_dense.cu): C[T, n_out] = A[T, k] W^T with 128 token rows per
// tile on the MMA's M side and 256 output features on its N side.  mode 0: feature FC (A = features, one weight
// matrix, one reduction range) -> z g-half = bf16(g * gain), ss[T][n_tiles] partial sums of squares.  mode 1:
// k / v (A = z; weight matrices W_k, W_v, each as its g-half and e-half columns: mapW[2*w + half]) ->
// y = rstd_g * (g half) + (e half), RoPE on k, bf16 into the caches.
struct DenseArgs {
  CUtensorMap mapA, mapW[4];
  int T, mode, n_w, n_tiles_per_w, n_out;
  int pair_waves;                                  // set by launch_umma_dense: waves of two-token-tile items (mode 0)
  int KB[2], a_koff[2];
  int h; float eps;
  const bf16* gain; bf16* z; long long ldz;       // mode 0 outputs
  float* ss; int ss_ld, ss_n;                      // [T][ss_ld] partial sums of squares (ss_n of them per row)
  int Hkv, dh; const float2* rope_tab; bf16* k_cache; bf16* v_cache; long long P_cap;
  int B; int seq_off[33]; int seq_P[32];          // packed row t of sequence b sits at position seq_P[b] + t - seq_off[b]
  int* status;
};
cudaError_t launch_umma_dense(const DenseArgs& a, int n_sm, cudaStream_t st);
// to be launched right after the feature FC of the same pass (see the kernel)
cudaError_t launch_prefill_embed(const int32_t* tokens, int T, int vocab, const bf16* embed, const bf16* gain_e, int h, float eps,
                                 bf16* z, long long ldz, int n_sm, cudaStream_t st);

// Self-test of the bounded waits (selftest.cu): a wait of `limit` tries on a barrier nobody signals; on expiry the
// status word becomes DEV_TIMEOUT.  ticket != NULL: one ticket is taken on that counter first.
cudaError_t launch_bounded_wait_probe(int limit, int* status, int* ticket, cudaStream_t st);

// 2-D bf16 tensor map [outer][inner] (row stride ld_bytes), box {box_inner, box_outer}, 128-byte swizzle, zero fill.
cudaError_t tmap_encode_bf16(CUtensorMap* m, const void* base, unsigned long long inner, unsigned long long outer,
                             unsigned long long ld_bytes, unsigned box_inner, unsigned box_outer);
// hi + lo activation buffers (lo = hi + pair_bytes) as one 3-D map; a box of box_rows tokens arrives as (hi, lo) row pairs.
cudaError_t tmap_encode_bf16_pair(CUtensorMap* m, const void* hi, unsigned long long pair_bytes, unsigned long long inner,
                                  unsigned long long rows, unsigned long long ld_bytes, unsigned box_rows);

// (cos, sin) table of RoPE for positions 0 .. n_pos-1 (once, at init)
cudaError_t launch_rope_table(float2* tab, int n_pos, int dh, float theta, cudaStream_t st);
// Copies the <mask> row into every z row (b, r) with r >= F (when the batch size or F changes)
struct FreshOffsets { int v[33]; };   // prefix sums of the per-sequence fresh counts
cudaError_t launch_fill_mask_rows(bf16* z_hi, bf16* z_lo, const bf16* zmask_hi, const bf16* zmask_lo, int B, int K,
                                  const FreshOffsets& foff, int width, cudaStream_t st);
// z row of the <mask> rows and the 1/rms of its g half (once, at init)
// feat_in = 0: g [n_fresh][h] given by the caller; writes what the feature FC's prologue and epilogue write.
cudaError_t launch_prefused_rows(const EpiArgs& e, const bf16* g, int n_fresh, cudaStream_t st);
cudaError_t launch_mask_row(const bf16* mask_vec, const bf16* norm_g, const bf16* norm_e, int h, float eps, bf16* z_hi,
                            bf16* z_lo, float* rstd_mask, float* mask_res, cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// Split-KV grouped-query attention over the cache (rows 0 .. P_b-1) and the step's new rows + combine.
// ---------------------------------------------------------------------------------------------
struct AttnParams {
  int B, K, Hq, Hkv, dh;
  const int32_t* seq_lens;
  const bf16* q_hi; const bf16* q_lo;      // [B,Hq,K,dh]
  const bf16* k_new; const bf16* v_new;    // [B,Hkv,16,dh] hi rows 0..7, lo rows 8..15
  const bf16* k_cache; const bf16* v_cache; long long P_cap;
  int chunk_keys;       // keys per CTA (multiple of 64)
  float* o_part;        // [sum_b chunks_b, Hkv, 64, dh]
  float* ml_part;       // [sum_b chunks_b, Hkv, 64, 2]
  bf16* a_hi; bf16* a_lo;  // [M, Hq*dh]
};
struct AttnArgs {
  AttnParams p;
  int chunk_base[33];  // prefix sums of chunks per sequence (cache chunks + 1 new-rows chunk)
};
// The tensor-core split kernel (attn_umma.cu, d_h = 128): tensor maps over q_hi / q_lo [B*Hq*K][128] (boxes of 16
// rows x 64 columns), the caches [B*Hkv*P_cap][128] and the new rows' side tiles [B*Hkv*16][128] (64 x 64).
struct AttnUmmaMaps { CUtensorMap mapQhi, mapQlo, mapK, mapV, mapKn, mapVn; };
struct AttnUmmaArgs {
  AttnArgs a;
  CUtensorMap mapQhi, mapQlo, mapK, mapV, mapKn, mapVn;
  int* status;
};
cudaError_t attn_umma_setup();  // once per device
cudaError_t launch_attn_umma_split(const AttnUmmaArgs& a, int max_chunks, cudaStream_t st);
cudaError_t attention_setup();  // once per device: opt in to the kernels' dynamic shared memory
// seq_lens_host: the same lengths on the host (sizes the grid and the partial layout); B <= 32.  With `maps`
// (d_h = 128, batches with a few thousand key tiles) the split runs on the tcgen05 kernel, otherwise on the warp-MMA one
// that a single sequence's few chunks are faster on; the combine is the same.
cudaError_t launch_attention(const AttnParams& p, const int* seq_lens_host, const AttnUmmaMaps* maps, int* status, cudaStream_t st);
// which split kernel launch_attention picks, and the chunk length that suits the tcgen05 one (0: none fits pairs_cap)
bool attn_uses_umma(int B, int Hkv, int dh, const int* seq_lens_host, bool have_maps);
int attn_umma_chunk_keys(int B, int Hkv, const int* seq_lens_host, int n_sm, int pairs_cap);

// ---------------------------------------------------------------------------------------------
// LM head with fused log-softmax / top-k partials, and the merge that finishes them.
// ---------------------------------------------------------------------------------------------
struct LmParams {
  StreamArgs s;  // unused by the LM-head kernels (kept zero)
  const bf16* W; int V; int Kd;
  const bf16* x_hi; const bf16* x_lo; long long ldx; int M; int K;  // token m = b*K + r
  const float* ss_in; int ss_tiles; int ss_mp; float rms_eps;  // final RMSNorm's 1/rms, applied to the logits
  int topk; float inv_temp; int gumbel; uint32_t seed_lo, seed_hi, step; float eps_logit;
  int grid;
  float* logits_out;       // nullable [M,V]
  float* part_stats;       // [grid][MP][2]  (max, sum exp)
  float* part_key; float* part_y; int32_t* part_id;  // [grid][MP][32]
  int32_t* out_ids; float* out_slogit;  // [M, topk]
};
// The LM head for up to 32 token rows (p.grid CTAs, at most one per SM so that all of them are resident at once).
// pieces: [grid][128][MP] fp32 partial logits of tiles cut between CTAs; flags: [grid] ints, a CTA's piece is
// complete when its flag equals `tag` (a value no earlier launch used).
struct LmUmmaArgs {
  LmParams p;
  CUtensorMap mapW, mapXhi, mapXlo;
  int KB; long long U;
  float* pieces; int* flags; int tag;
  int* status;
  unsigned long long* bound;   // lm_head_dense_kernel: [128 token rows][kLmBoundSlots] shared lower bounds (tag << 32 | ordered key)
};
constexpr int kLmBoundSlots = 40;   // topk + 7 of them are used
// units of work of an LM-head launch; its grid must not exceed them (nor the SM count: the CTAs wait on one another)
long long lm_head_units(int V, int Kd, bool dense);
cudaError_t launch_lm_head_umma(const LmParams& p, const CUtensorMap& mapW, const CUtensorMap& mapX,
                                float* pieces, int* flags, int tag, int* status, cudaStream_t st);
// The LM head for 33..128 token rows with the operands swapped (token rows on the MMA's M side; lm_head.cu).
// mapW256: the weight matrix with boxes of 256 rows; mapXhi / mapXlo: 2-D maps [M][Kd], boxes of 128 rows;
// pieces: [grid][128][256] fp32.  The per-CTA results are laid out for MP = 128 token rows.
// bound: kLmBoundSlots 64-bit words per token row, zero before the first launch; tags must differ between launches.
cudaError_t launch_lm_head_dense(const LmParams& p, const CUtensorMap& mapW256, const CUtensorMap& mapXhi, const CUtensorMap& mapXlo,
                                 float* pieces, int* flags, int tag, int* status, unsigned long long* bound, cudaStream_t st);
cudaError_t topk_merge_setup(int max_grid);  // once per device
cudaError_t launch_topk_merge(const LmParams& p, cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// Forward attention under the prefix-shared training mask (train_attn.cu).  head_dim = 128.
// ---------------------------------------------------------------------------------------------
// Prefix positions whose masked blocks share one 128-row query tile.
__host__ __device__ inline int train_attn_positions_per_tile(int d) { return 128 / d; }
struct TrainAttnArgs {
  CUtensorMap mapQ, mapK, mapV;   // [B*H*L][128] bf16, boxes of 128 (Q) / 64 (K, V) rows x 64 columns
  int B, Hq, Hkv, prompt_len, draft_len, n_clean_tiles;
  int seq_len[64];             // valid prompt slots per sequence
  float scale_log2e;           // log2(e) / sqrt(head_dim)
  bf16* out;                   // [B][Hq][L][128]
  int* status;                 // may be null
};
cudaError_t launch_train_attn(const TrainAttnArgs& a, cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// N-gram hash table + tree pruning.
// ---------------------------------------------------------------------------------------------
// Open addressing over buckets of eight rows.  A row lives in the bucket its key hashes to, or -- when that one was
// full at build time -- in the next bucket with room (linear probing over buckets, the longest displacement recorded
// as max_probe).  Per bucket there are eight 16-bit fingerprints of the keys in one 16-byte word (0 = empty slot) and,
// in a second array, the eight {key, score} slots.  A lookup reads the fingerprint word -- ONE 16-byte request -- and a
// slot only where a fingerprint matches: a miss ends at a word with an empty slot and no match, one request in all.
// (The sweep makes ~10^5 lookups per tree, every lane of a warp in another line of the table: what bounds it is the
// number of such scattered requests an SM can issue, not their latency.  Four requests per lookup -- a bucket's eight
// full keys -- took 5.2 us per round of lookups; probing 16-byte slots one after the other took as long.)
struct NgramSlot { unsigned long long key; float score; uint32_t pad; };  // 16 bytes
struct NgramTable { const uint4* fp; const NgramSlot* slots; uint32_t mask; uint32_t max_probe; };   // mask: buckets - 1
__host__ __device__ inline uint32_t ngram_fingerprint(unsigned long long hash) {
  const uint32_t f = (uint32_t)(hash >> 48);
  return f == 0u ? 1u : f;     // 0 marks an empty slot
}
// The same rows as child lists (Appendix C).  Every list is a run of {key, payload} slots in ascending key order:
//   2-gram context b   -> bi_ent[bi_off[b] .. bi_off[b+1])             {next token, score bits}
//   first token a      -> tri_node[tri_off[a] .. tri_off[a+1])         {second context token b, first child}, then a
//                                                                      sentinel {0x7fffffff, end of the last node's children}
//   3-gram context j   -> tri_ent[tri_node[j].y .. tri_node[j+1].y)    {next token, score bits}
// A region may end in slots with key 0xffffffff (alignment filler).  A list of more than kTrieLongList slots is
// long: its region starts on a 64-byte boundary with nb8 / 8 bitmap blocks of 16 words -- {entries before this
// block, 480 bits: token 480 * block + r is in the list} -- followed by the list, so that the entry of token t is
// slot nb8 + (entries before its block) + (set bits below r) of the region.  Regions of kTrieLongList + 7 slots or
// fewer are short lists; anything larger starts with the bitmap.
constexpr int kTrieLongList = 1016;
struct NgramTrie { const uint32_t* bi_off; const uint2* bi_ent; const uint32_t* tri_off; const uint2* tri_node; const uint2* tri_ent; uint32_t nb8; };
struct NgramTrieOwned { uint32_t* bi_off; uint2* bi_ent; uint32_t* tri_off; uint2* tri_node; uint2* tri_ent; size_t bytes; };
// Host rows -> device child lists (rows must have been validated; 3-gram rows are skipped when ngram_order < 3;
// of duplicate rows the first wins).  Synchronous; on failure everything allocated so far is released.
cudaError_t ngram_trie_build(const unsigned char* order, const int32_t* c0, const int32_t* c1, const int32_t* nx, const float* score,
                             long long n_rows, int vocab, int ngram_order, NgramTrieOwned* out);
void ngram_trie_free(NgramTrieOwned* t);

struct TreeParams {
  int B, K, topk, beam, budget, first_row, n_levels, ngram_order, vocab;
  unsigned char first_rows[32];   // per sequence: first logit row = level 0; levels = min(n_levels, K - first row)
  const int32_t* ids; const float* slogit; const int32_t* ctx_tail;
  NgramTable table;
  NgramTrie trie;   // used instead of `table` when trie.bi_off != nullptr
  float* sg;   // [B][tree_sg_floats] dense s_ng table of the hash layout (workspace, written by ngram_sweep_kernel)
  float* bg;   // [B][topk + (n_levels-1)*topk^2] bigram scores of the trie layout (workspace, written by trie_sweep_kernel)
  uint2* cx;   // [B][1 + topk + (n_levels-2)*topk^2] child ranges of the 3-gram contexts (trie layout only)
  float wl[8]; float wv[8]; float wn; float miss;
  int32_t* tokens; int32_t* parents; int32_t* depth; uint8_t* mask; int32_t* n_nodes; float* scores;
  int* status;
};
cudaError_t tree_setup(int topk, int beam, int budget, int max_levels);  // once per device
// Position ids and root-to-leaf paths of the trees (verification inputs); budget <= 64.
cudaError_t launch_verify_inputs(int B, int budget, int max_levels, const int32_t* parents, const int32_t* depth, const int32_t* n_nodes,
                                 const int32_t* root_pos, int32_t* position_ids, int32_t* retrieve, int32_t* n_leaves, cudaStream_t st);
size_t tree_smem_bytes(int topk, int beam, int budget, int n_levels);
size_t tree_sg_floats(int topk, int levels);   // floats per sequence of TreeParams::sg
cudaError_t launch_tree(const TreeParams& p, cudaStream_t st);

// key packing shared by the host-side table builder and the device lookup
__host__ __device__ inline unsigned long long ngram_key(int order, int c0, int c1, int next) {
  const unsigned long long a = (order == 3) ? (unsigned long long)(uint32_t)(c0 + 1) : 0ull;
  return ((unsigned long long)(order == 3 ? 1 : 0) << 63) | (a << 42) |
         ((unsigned long long)(uint32_t)(c1 + 1) << 21) | (unsigned long long)(uint32_t)(next + 1);
}
__host__ __device__ inline unsigned long long ngram_hash(unsigned long long x) {
  x ^= x >> 30; x *= 0xbf58476d1ce4e5b9ull;
  x ^= x >> 27; x *= 0x94d049bb133111ebull;
  x ^= x >> 31;
  return x;
}

}  // namespace dart
