// Internal interface between the C-ABI layer (api.cu) and the kernel translation units.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace dart {

typedef __nv_bfloat16 bf16;

// ---------------------------------------------------------------------------------------------
// Weight-streaming small-M GEMM, "rows" mode:  part = W[rows, Kd] * x[M, Kd]^T, split over the
// flattened (128-row tile, 64-wide k-step) space so that every CTA streams the same number of
// weight bytes.  A CTA writes one fp32 partial per tile it touches; a finalize kernel sums the
// partials of a tile in CTA order (deterministic) and applies the op that follows the GEMM.
// ---------------------------------------------------------------------------------------------
struct GemmSeg {
  const bf16* W;  // [rows, Kd] row-major
  int rows;       // multiple of 16
  int tile0;      // index of this segment's first 128-row tile in the launch
};

struct GemmPlan {
  int nseg;
  GemmSeg seg[3];
  int Kd;         // reduction length, multiple of 16
  int SK;         // ceil(Kd / 64) k-steps per tile
  int n_tiles;    // 128-row tiles over all segments
  int grid;       // CTAs
  int slots;      // max tiles a CTA touches
  long long U;    // n_tiles * SK
  int* d_tile_clo;  // DEVICE [n_tiles] first CTA contributing to a tile
  int* d_tile_chi;  // DEVICE [n_tiles] last CTA contributing to a tile
};

// What a finalize kernel needs to sum a tile's partials.
struct PartView {
  const float* part;  // [grid][slots][128][MP]
  const int* clo;
  const int* chi;
  int SK;
  long long U;
  int G;
  int slots;
  int MP;  // padded token count (8, 32 or 128)
};

inline PartView make_view(const GemmPlan& p, const float* part, int MP) {
  PartView v;
  v.part = part; v.clo = p.d_tile_clo; v.chi = p.d_tile_chi; v.SK = p.SK; v.U = p.U; v.G = p.grid;
  v.slots = p.slots; v.MP = MP;
  return v;
}

__host__ __device__ inline int padded_tokens(int M) { return M <= 8 ? 8 : (M <= 32 ? 32 : 128); }

// x_hi/x_lo: bf16 [>=M, ldx] activations (lo may be NULL: plain bf16 input).  M valid tokens.
cudaError_t launch_gemm_rows(const GemmPlan& plan, const bf16* x_hi, const bf16* x_lo, long long ldx, int M,
                             float* part, cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// Finalize kernels (one CTA per token row).
// ---------------------------------------------------------------------------------------------
struct StageParams {  // S0: z = [RMSNorm(g); RMSNorm(e)], residual = g
  PartView fc;        // FC partials, token index = b*F + r (only when F > 0)
  int B, K, F, h;
  const int32_t* tokens;  // [B,F]
  int vocab;
  const bf16* embed; const bf16* mask_vec; const bf16* norm_g; const bf16* norm_e;
  float eps;
  float* res;      // [M, h] fp32 residual stream (out)
  bf16* z_hi; bf16* z_lo;  // [M, 2h]
};
cudaError_t launch_stage_inputs(const StageParams& p, cudaStream_t st);

struct QkvParams {  // S1 epilogue: RoPE + cache write
  PartView qkv;     // rows: [q heads | k heads | v heads] (three segments)
  int q_tile0, k_tile0, v_tile0;
  int B, K, Hq, Hkv, dh;
  const int32_t* seq_lens;
  float rope_theta;
  int F;             // rows r < F are fresh: their k, v are appended to the cache at P_b + r
  bf16* q_hi; bf16* q_lo;        // [B, Hq, K, dh] post-RoPE queries as hi + lo
  bf16* k_new; bf16* v_new;      // [B, Hkv, 16, dh]: rows 0..7 hi parts of the K new rows, rows 8..15 lo parts
  bf16* k_cache; bf16* v_cache;  // [*, Hkv, P_cap, dh]
  long long P_cap;
};
cudaError_t launch_qkv_finalize(const QkvParams& p, cudaStream_t st);

struct ResNormParams {  // x_out = res + sum(parts); n = RMSNorm(x_out) * gamma
  PartView proj;
  int M, h;
  const bf16* gamma; float eps;
  float* res;          // [M,h] in/out (updated in place)
  bf16* n_hi; bf16* n_lo;  // [M,h]
};
cudaError_t launch_res_norm(const ResNormParams& p, cudaStream_t st);

struct GateUpParams {  // u = SiLU(gate) * up
  PartView gu;  // two segments: gate rows then up rows
  int up_tile0;
  int M, I;
  bf16* u_hi; bf16* u_lo;  // [M, I]
};
cudaError_t launch_gate_up(const GateUpParams& p, cudaStream_t st);

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
cudaError_t attention_setup();  // once per device: opt in to the kernel's dynamic shared memory
// seq_lens_host: the same lengths on the host (sizes the grid and the partial layout); B <= 32
cudaError_t launch_attention(const AttnParams& p, const int* seq_lens_host, cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// LM head with fused log-softmax / top-k partials, and the merge that finishes them.
// ---------------------------------------------------------------------------------------------
struct LmParams {
  const bf16* W; int V; int Kd;
  const bf16* x_hi; const bf16* x_lo; long long ldx; int M; int K;  // token m = b*K + r
  int topk; float inv_temp; int gumbel; uint32_t seed_lo, seed_hi, step; float eps_logit;
  int grid;
  float* logits_out;       // nullable [M,V]
  float* part_stats;       // [grid][MP][2]  (max, sum exp)
  float* part_key; float* part_y; int32_t* part_id;  // [grid][MP][32]
  int32_t* out_ids; float* out_slogit;  // [M, topk]
};
cudaError_t launch_lm_head(const LmParams& p, cudaStream_t st);
cudaError_t topk_merge_setup(int max_grid);  // once per device
cudaError_t launch_topk_merge(const LmParams& p, cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// N-gram hash table + tree pruning.
// ---------------------------------------------------------------------------------------------
struct NgramSlot { unsigned long long key; float score; uint32_t pad; };  // 16 bytes; key 0 = empty
struct NgramTable { const NgramSlot* slots; uint32_t mask; uint32_t max_probe; };

struct TreeParams {
  int B, K, topk, beam, budget, first_row, n_levels, ngram_order;
  const int32_t* ids; const float* slogit; const int32_t* ctx_tail;
  NgramTable table;
  float wl[8]; float wv[8]; float wn; float miss;
  int32_t* tokens; int32_t* parents; int32_t* depth; uint8_t* mask; int32_t* n_nodes; float* scores;
  int* status;
};
cudaError_t tree_setup(int topk, int beam, int budget, int max_levels);  // once per device
size_t tree_smem_bytes(int topk, int beam, int budget, int n_levels);
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
