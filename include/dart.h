/*
 * dart.h -- C ABI of the B200 (sm_100a) implementation of DART's drafting step.
 *
 * One call of dart_draft_step followed by one call of dart_build_tree is one "draft step":
 * target hidden states -> one draft decoder layer over the prefix KV cache plus K query rows
 * -> LM head -> per-position log-softmax + top-k -> N-gram-scored tree pruning -> a
 * fixed-budget draft token tree (token ids, parents, tree-attention mask).
 *
 * Conventions
 *   - Every pointer is labelled HOST or DEVICE.  Device buffers are caller-owned unless stated.
 *   - bf16 tensors are row-major with the last index fastest; weight matrices are [out, in];
 *     weight pointers and `feats` must be 32-byte aligned and their row strides multiples of 16 bytes
 *     (they are read by TMA tile loads, or by 256-bit loads in the fallback kernels), every other device
 *     pointer 16-byte aligned.
 *   - All GPU work is enqueued on the CUDA stream passed as `void* cuda_stream` (a cudaStream_t;
 *     NULL = the legacy default stream).  dart_draft_step and dart_build_tree do not
 *     synchronise, allocate, or copy between host and device.
 *   - Return value: DART_OK (0) or a negative dart_status.  Argument errors are reported
 *     synchronously and enqueue nothing.  Errors that only the device can detect (a lookup
 *     that ran past its probe bound, a bounded wait on a barrier or on another CTA's flag that ran
 *     out) set a status word read by dart_last_device_status; the kernels never wait without a limit.
 *   - One handle may be used from one host thread and one stream at a time.
 *   - There is no CPU fallback: on a machine without an sm_100 device dart_draft_init fails.
 */
#ifndef DART_H_
#define DART_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum dart_status {
  DART_OK = 0,
  DART_ERR_INVALID_ARG = -1,      /* NULL/misaligned pointer, shape the kernels do not support */
  DART_ERR_UNSUPPORTED_ARCH = -2, /* current device is not compute capability 10.x */
  DART_ERR_CUDA = -3,             /* a CUDA runtime call failed; see dart_last_cuda_error */
  DART_ERR_CAPACITY = -4,         /* batch > max_batch, or prefix + K > max_prefix */
  DART_ERR_TIMEOUT = -5,          /* a bounded device-side loop gave up (device status word) */
  DART_ERR_INTERNAL = -6
} dart_status;

typedef struct dart_handle dart_handle; /* opaque; owns workspace + the device N-gram table */

/*
 * Shapes and hyper-parameters, fixed for the lifetime of a handle.
 * Layer shapes follow Appendix B ("hyperparameters ... aligned with the target model");
 * topk/beam/tree_budget and the Combine weights are Appendix D's k_i, w, theta+1, w_ng,
 * 0.9^level, (level+1)^-0.7.
 */
typedef struct dart_config {
  uint32_t struct_size;  /* = sizeof(dart_config); guards against layout mismatch */
  int32_t hidden;        /* h; multiple of 64 */
  int32_t n_q_heads;     /* H_q */
  int32_t n_kv_heads;    /* H_kv; H_q % H_kv == 0 and (H_q/H_kv)*K <= 64 */
  int32_t head_dim;      /* d_h: 64 or 128 */
  int32_t mlp_inter;     /* I; multiple of 16 */
  int32_t vocab;         /* V; multiple of 16, < 2^21 */
  int32_t feat_in;       /* width of the concatenated target features (3h); multiple of 16.  0: the caller fuses the
                            features itself and passes g [.., hidden] as `feats`; w_fc is unused, no prefill */
  int32_t max_batch;     /* sequences per call; <= 32 and max_batch * K <= 128 */
  int32_t max_prefix;    /* P_cap: rows per sequence in the caller's KV cache */
  int32_t K;             /* query rows per sequence = future positions d (Section 3.2); 1..8 */
  int32_t topk;          /* k_i: candidates kept per position, 1..32 (Appendix D: 25) */
  int32_t beam;          /* w: beam width, 1..32 (Appendix D: 20) */
  int32_t tree_budget;   /* nodes in the output tree including the root, 2..64 (theta + 1 = 60) */
  int32_t ngram_order;   /* 2 or 3 (Appendix C: 3) */
  float rope_theta;      /* RoPE base (1e6) */
  float rms_eps;         /* RMSNorm epsilon (1e-6) */
  float w_ng;            /* Combine: N-gram weight (0.5) */
  float logit_decay;     /* Combine: w_logit = logit_decay^level (0.9) */
  float level_exp;       /* Combine: w_level = (level+1)^-level_exp (0.7) */
  float eps_logit;       /* epsilon inside s_logit = log(softmax + eps) */
  float eps_ng;          /* epsilon of a missing N-gram: s_ng = log(eps_ng) */
  float temperature;     /* 0 = deterministic top-k; > 0 = Gumbel-top-k on logits / temperature */
  uint64_t philox_seed;  /* key of the Philox4x32-10 stream used when temperature > 0 */
  int32_t ngram_layout;  /* device layout of the N-gram: DART_NGRAM_HASH or DART_NGRAM_TRIE (Appendix C) */
  int32_t reserved0;     /* 0 */
} dart_config;

/*
 * Draft-model parameters (Appendix B "Trainable parameters": FC, decoder layer, LM head, mask
 * representation; the embedding is the target's).  DEVICE pointers to bf16, row-major
 * [out, in]; caller-owned, never written, must outlive the handle.
 */
typedef struct dart_weights {
  const void* w_fc;       /* [h, feat_in]   fusion of the three target layers' hidden states */
  const void* embed;      /* [V, h]         target embedding table (shifted token embedding) */
  const void* mask_vec;   /* [2h]           learned <mask> representation, stands for [g ; e] */
  const void* norm_g;     /* [h]            RMSNorm gain on g */
  const void* norm_e;     /* [h]            RMSNorm gain on e */
  const void* w_q;        /* [H_q*d_h, 2h]  */
  const void* w_k;        /* [H_kv*d_h, 2h] */
  const void* w_v;        /* [H_kv*d_h, 2h] */
  const void* w_o;        /* [h, H_q*d_h]   */
  const void* norm_post;  /* [h]            RMSNorm gain before the MLP */
  const void* w_gate;     /* [I, h] */
  const void* w_up;       /* [I, h] */
  const void* w_down;     /* [h, I] */
  const void* norm_final; /* [h]            RMSNorm gain before the LM head */
  const void* w_lm;       /* [V, h]         the drafter's own LM head */
} dart_weights;

/*
 * N-gram rows (Appendix C), HOST arrays of length n_rows, copied into a library-owned
 * device hash table by dart_draft_init.  Row i says: after context (ctx0[i], ctx1[i]) the
 * token next[i] has continuity score score[i] = log(Pr(next | context) + eps), Appendix D's
 * s_ng.  order[i] is 3 (trigram) or 2 (bigram; ctx0[i] ignored).  Of duplicate rows the first wins.
 */
#define DART_NGRAM_HASH 0 /* open-addressing table, one 16-byte slot per row at load <= 0.5: one probe per lookup */
#define DART_NGRAM_TRIE 1 /* child lists (Appendix C): the context's node is located once, its children are then
                             searched for every candidate; 8 bytes per row plus 8 per distinct 3-gram context */
typedef struct dart_ngram_host {
  int64_t n_rows;
  const uint8_t* order;
  const int32_t* ctx0;
  const int32_t* ctx1;
  const int32_t* next;
  const float* score;
} dart_ngram_host;

/*
 * Inputs of one forward pass (Section 3.2).  Per sequence b the K query rows are
 * r = 0..K-1 at absolute positions P_b + r, P_b = seq_lens[b]; rows r < n_fresh carry fresh
 * target features and the id of the token that follows them (shifted embedding), the rest
 * are <mask> rows.  The canonical step is n_fresh = 1: the last prefix position plus d-1 masks.
 * After a verification that accepted a different number of tokens per sequence the counts differ:
 * fresh_counts_host[b] = F_b then replaces n_fresh, and the fresh rows' features and token ids are
 * packed in sequence order (sequence 0's F_0 rows, then sequence 1's, ...).
 */
typedef struct dart_step_in {
  int32_t batch;          /* B <= max_batch */
  int32_t n_fresh;        /* F, 0..K (0: K mask rows, feats/tokens unused) */
  const void* feats;      /* DEVICE bf16 [B, F, feat_in]  (packed [sum F_b, feat_in] with fresh_counts_host); with
                             feat_in = 0 the fused features g, [B, F, hidden] */
  const int32_t* tokens;  /* DEVICE i32  [B, F] next-token ids, 0 <= id < V  (packed [sum F_b]) */
  const int32_t* seq_lens;      /* DEVICE i32 [B]  P_b: rows already in the cache */
  const int32_t* seq_lens_host; /* HOST   i32 [B]  same values; used for capacity checks and launch sizing */
  void* k_cache;          /* DEVICE bf16 [max_batch, H_kv, max_prefix, d_h], post-RoPE keys */
  void* v_cache;          /* DEVICE bf16, same layout.  The call appends the fresh positions' k, v: it writes
                             rows P_b .. P_b+F-1 of both caches and nothing else (the <mask> rows' k, v
                             are transient); the caller advances seq_lens.  Needs P_b + F <= max_prefix. */
  uint64_t step_counter;  /* Philox counter word; change it every call when temperature > 0 */
  const int32_t* fresh_counts_host; /* HOST i32 [B] per-sequence fresh-row counts F_b in 0..K, or NULL: every
                                       sequence has n_fresh.  With it the call appends rows P_b .. P_b+F_b-1. */
} dart_step_in;

/*
 * Outputs of one forward pass: Algorithm 1 lines 6-8 for every logit row.  Row r predicts
 * the token after position P_b + r (shifted logits); rows r >= max(F,1)-1 are the d logit
 * rows of Section 3.2, earlier rows are computed as well.
 */
typedef struct dart_step_out {
  int32_t* topk_ids;      /* DEVICE i32 [B, K, topk]  S_i, by selection value desc, ties lower id */
  float* topk_slogit;     /* DEVICE f32 [B, K, topk]  s_logit = log(softmax(logits/T) + eps_logit) */
  float* logits;          /* DEVICE f32 [B, K, V] or NULL.  Full logits (before 1/T), for checking only */
} dart_step_out;

/* Inputs of Algorithm 1 for B sequences. */
typedef struct dart_tree_in {
  int32_t batch;
  int32_t first_row;          /* first logit row used as level 0 (= max(F,1)-1) */
  int32_t n_levels;           /* d = number of levels, first_row + n_levels <= K */
  const int32_t* topk_ids;    /* DEVICE i32 [B, K, topk] as written by dart_draft_step */
  const float* topk_slogit;   /* DEVICE f32 [B, K, topk] */
  const int32_t* ctx_tail;    /* DEVICE i32 [B, 2]: the last two known tokens (c_-2, c_-1); -1 = absent */
  const int32_t* first_rows_host; /* HOST i32 [B] per-sequence first logit row (= max(F_b,1)-1), or NULL: first_row for
                                     all.  Sequence b then has min(n_levels, K - first_rows_host[b]) levels. */
} dart_tree_in;

/*
 * The pruned draft tree per sequence.  Slot 0 is the root (token c_-1, parent -1, depth 0);
 * slots 1..n_nodes-1 are the selected nodes by score descending.  parents[x] < x.
 * mask[x][y] = 1 iff y == x or y is an ancestor of x (the tree-attention mask).
 * Unused slots: token -1, parent -1, depth -1, mask row 0.
 */
typedef struct dart_tree_out {
  int32_t* tokens;   /* DEVICE i32 [B, tree_budget] */
  int32_t* parents;  /* DEVICE i32 [B, tree_budget] */
  int32_t* depth;    /* DEVICE i32 [B, tree_budget] */
  uint8_t* mask;     /* DEVICE u8  [B, tree_budget, tree_budget] */
  int32_t* n_nodes;  /* DEVICE i32 [B] */
  float* scores;     /* DEVICE f32 [B, tree_budget] or NULL: the (ancestor-clamped) node scores */
} dart_tree_out;

/*
 * Create a handle (Section 3.2 + Section 4 set-up): validates cfg, records the weight
 * pointers, builds the device N-gram hash table from the host rows (ngram may be NULL or
 * empty: every lookup then misses), allocates the workspace (the only allocation the library
 * ever makes) and precomputes Appendix D's per-level weights.  Synchronous.
 * Errors: INVALID_ARG, UNSUPPORTED_ARCH, CUDA.  *out is NULL on failure.
 */
int dart_draft_init(const dart_config* cfg, const dart_weights* weights, const dart_ngram_host* ngram,
                    dart_handle** out);

/*
 * One forward pass of the draft layer and LM head with fused log-softmax/top-k
 * (Section 3.2; Algorithm 1 lines 6-8; Appendix D s_logit).  Asynchronous on `cuda_stream`.
 * Errors: INVALID_ARG (NULL pointers, a fresh-row count out of range), CAPACITY (batch > max_batch or
 * seq_lens_host[b] + F_b > max_prefix).
 */
int dart_draft_step(dart_handle* h, const dart_step_in* in, const dart_step_out* out, void* cuda_stream);

/*
 * Continuity-aware tree pruning (Algorithm 1, Appendix D) for B sequences, one thread block
 * per sequence.  Asynchronous on `cuda_stream`.  Bit-exact with a sequential fp32 evaluation
 * of Algorithm 1 that breaks ties by generation order.  Errors: INVALID_ARG, CAPACITY.
 */
int dart_build_tree(dart_handle* h, const dart_tree_in* in, const dart_tree_out* out, void* cuda_stream);

/*
 * One whole draft step for a caller whose step inputs and tree outputs live in HOST memory (Section 3.2 followed by
 * Algorithm 1, as one call): copies `in_bytes` from `in_host` to `in_dev`, runs dart_draft_step(in, out) and
 * dart_build_tree(tree_in, tree_out), copies `out_bytes` from `out_dev` to `out_host` and waits for `cuda_stream`.
 * The device pointers of `in` / `tree_in` (feats, tokens, seq_lens, ctx_tail) are expected to point into
 * [in_dev, in_dev + in_bytes) and those of `tree_out` into [out_dev, out_dev + out_bytes): the layout inside the two
 * buffers is the caller's.  Host buffers should be page-locked (pageable memory works, more slowly).  All buffers
 * are caller-owned; nothing is allocated.  Synchronous: on return the tree is in `out_host`.
 * Errors: those of the two calls; INVALID_ARG for a NULL buffer with a non-zero size; CUDA if a copy or the wait fails.
 */
typedef struct dart_host_io {
  const void* in_host;   /* HOST   step inputs, in_bytes */
  void* in_dev;          /* DEVICE their home on the device */
  size_t in_bytes;
  const void* out_dev;   /* DEVICE tree outputs, out_bytes */
  void* out_host;        /* HOST   where the caller reads them */
  size_t out_bytes;
} dart_host_io;
int dart_draft_step_host(dart_handle* h, const dart_host_io* io, const dart_step_in* in, const dart_step_out* out,
                         const dart_tree_in* tree_in, const dart_tree_out* tree_out, void* cuda_stream);

/* Free the workspace and the N-gram table.  The caller's buffers are untouched. */
int dart_draft_destroy(dart_handle* h);

/* Device-side status word since the last call of this function: DART_OK or DART_ERR_TIMEOUT.
 * Synchronises `cuda_stream`.  After DART_ERR_TIMEOUT the outputs of the calls since the previous check are void;
 * the call has then also cleared the handle's internal work counters (a kernel that gives up on a wait leaves
 * them half counted), so the handle stays usable: the next dart_draft_step starts from a clean state. */
int dart_last_device_status(dart_handle* h, void* cuda_stream);

/*
 * Self-test of the time-out path (the paper has no counterpart).  Every device-side wait of this library is
 * bounded: when it runs out the kernel records DART_ERR_TIMEOUT in the handle's status word and returns.  This call
 * enqueues a one-block kernel that runs exactly that path on purpose -- a wait of `spin_limit` tries (1 .. 100000,
 * each at most 2 microseconds) on a barrier that nothing signals -- so that a caller (or a test) can see the error
 * arrive through dart_last_device_status and the handle recover.  leave_ticket != 0 additionally leaves one work
 * counter of the QKV projection half counted, as a kernel that gave up mid-way would.  Faults nothing, hangs nothing.
 * Asynchronous on `cuda_stream`.  Errors: INVALID_ARG, CUDA.
 */
int dart_selftest_bounded_wait(dart_handle* h, int32_t spin_limit, int32_t leave_ticket, void* cuda_stream);

/* The cudaError_t (as int) behind the last DART_ERR_CUDA of this handle; with h = NULL, of the last call that has no
 * handle (dart_draft_init, dart_train_attention_fwd, dart_topk_rows_noalloc). */
int dart_last_cuda_error(const dart_handle* h);

/* Human-readable name of a dart_status. */
const char* dart_status_string(int status);

/* Bytes of device workspace a handle for `cfg` allocates (excluding the N-gram table); 0 if cfg is invalid. */
size_t dart_workspace_bytes(const dart_config* cfg);

/*
 * Forward attention under the prefix-shared training mask (Section 3.3 "Prefix-shared masked training", Appendix B).
 * A packed row has L = prompt_len * (1 + draft_len) slots: prompt_len clean positions, then one block of draft_len
 * masked positions per prefix position n.  Clean slot q reads clean slots <= q; block n reads clean slots 0..n and
 * its own slots up to the reading one; blocks never read each other.  Slots past seq_lens_host[b] (clean slots >= it,
 * blocks of prefix positions >= it) read nothing and give zero rows.  Grouped-query heads: head j reads KV head
 * j / (n_q_heads / n_kv_heads).  Softmax scale 1 / sqrt(head_dim).
 */
typedef struct dart_train_attn_in {
  int32_t batch;             /* 1..64 */
  int32_t n_q_heads, n_kv_heads;
  int32_t head_dim;          /* 128 */
  int32_t prompt_len;        /* clean positions per packed row, >= 1 */
  int32_t draft_len;         /* d, 1..16 */
  const void* q;             /* DEVICE bf16 [batch, n_q_heads, L, head_dim], 16-byte aligned; RoPE already applied */
  const void* k;             /* DEVICE bf16 [batch, n_kv_heads, L, head_dim] */
  const void* v;             /* DEVICE bf16 [batch, n_kv_heads, L, head_dim] */
  const int32_t* seq_lens_host; /* HOST [batch]: valid prompt slots, 0..prompt_len */
  void* out;                 /* DEVICE bf16 [batch, n_q_heads, L, head_dim]; every row is written */
  int32_t* status;           /* DEVICE, may be NULL: set to a negative code if a bounded wait inside the kernel ran out */
} dart_train_attn_in;

/*
 * Enqueues the attention on `cuda_stream` (one kernel; no workspace, no handle).  Errors: INVALID_ARG (NULL or
 * misaligned pointers, sizes out of range, head_dim != 128), UNSUPPORTED_ARCH, CUDA.
 */
int dart_train_attention_fwd(const dart_train_attn_in* in, void* cuda_stream);

/* Bytes of device memory the N-gram of this handle occupies in its layout (0 without an N-gram or handle). */
size_t dart_ngram_bytes(const dart_handle* h);

/* Number of kernels one dart_draft_step / dart_build_tree call enqueues for this batch size
 * (used by benchmarks to report launch counts). */
int dart_step_launch_count(const dart_handle* h, int batch, int n_fresh);

/*
 * Verification inputs of a draft tree (Section 3, Figure 2: the tree is verified by the target model in one
 * forward pass with tree attention; the attention mask is dart_tree_out.mask).  The paper names the step, not
 * its encoding; this one is the usual pair: node x sits at absolute position root_pos[b] + depth[x] (root_pos =
 * position of the root token c_-1), and a candidate continuation is a root-to-leaf path given as the slots of its
 * nodes.  retrieve row j = path of the j-th leaf (leaves in ascending slot order), root first, padded with -1;
 * rows past n_leaves and position ids of unused slots are -1.  One small kernel, asynchronous on `cuda_stream`.
 * Errors: INVALID_ARG, CAPACITY (batch > max_batch).
 */
typedef struct dart_verify_in {
  int32_t batch;
  int32_t max_levels;         /* columns of retrieve minus one: >= the deepest node's depth (K is always enough) */
  const int32_t* parents;     /* DEVICE i32 [B, tree_budget] as written by dart_build_tree */
  const int32_t* depth;       /* DEVICE i32 [B, tree_budget] */
  const int32_t* n_nodes;     /* DEVICE i32 [B] */
  const int32_t* root_pos;    /* DEVICE i32 [B] absolute position of each sequence's root token */
} dart_verify_in;
typedef struct dart_verify_out {
  int32_t* position_ids;      /* DEVICE i32 [B, tree_budget] */
  int32_t* retrieve;          /* DEVICE i32 [B, tree_budget, max_levels + 1] */
  int32_t* n_leaves;          /* DEVICE i32 [B] */
} dart_verify_out;
int dart_tree_verify_inputs(dart_handle* h, const dart_verify_in* in, const dart_verify_out* out, void* cuda_stream);

/*
 * Draft-side prefill (Section 3.2: the draft layer attends over its own KV cache of the prefix, which has to
 * exist before the first drafting step).  A single layer's keys and values depend on nothing but the layer's
 * input, so building the cache for new prefix positions needs no attention: for every new row the call
 * computes z = [RMSNorm(W_fc f) ; RMSNorm(E[token])], k = RoPE(W_k z) and v = W_v z at the row's absolute
 * position and stores them.  Sequence b gets new_rows_host[b] rows at positions seq_lens_host[b] ..; their
 * features and next-token ids are packed in sequence order.  The caller then advances its sequence lengths and
 * runs dart_draft_step as usual (whose own fresh rows are appended by that call).  No logits are produced.
 * Asynchronous on `cuda_stream`; the packed rows are processed in passes of up to 4096 rows (three kernel launches
 * per pass: token embeddings, feature FC, k / v projection), a sequence may straddle two passes.
 * Errors: INVALID_ARG (also with feat_in = 0: the prefill needs the fusion matrix), CAPACITY (batch > max_batch or
 * seq_lens_host[b] + new_rows_host[b] > max_prefix).
 */
typedef struct dart_prefill_in {
  int32_t batch;                  /* B <= max_batch */
  const void* feats;              /* DEVICE bf16 [sum N_b, feat_in], 32-byte aligned */
  const int32_t* tokens;          /* DEVICE i32  [sum N_b] id of the token that follows each row */
  const int32_t* seq_lens_host;   /* HOST i32 [B] rows already in the cache */
  const int32_t* new_rows_host;   /* HOST i32 [B] N_b >= 0 rows to add */
  void* k_cache;                  /* DEVICE bf16 [max_batch, H_kv, max_prefix, d_h]; rows P_b .. P_b+N_b-1 are written */
  void* v_cache;                  /* DEVICE bf16, same layout */
} dart_prefill_in;
int dart_draft_prefill(dart_handle* h, const dart_prefill_in* in, void* cuda_stream);

/*
 * Measurement aid (the paper has no counterpart): the next dart_draft_step (stages 0..7) or
 * dart_build_tree (stage 8) records the caller-owned CUDA events `start_event` / `stop_event`
 * (cudaEvent_t handles) on the stream immediately before and after the kernels of `stage`,
 * then forgets them.  Stages: 0 feature FC + input staging, 1 QKV + RoPE, 2 attention,
 * 3 o_proj + norm, 4 gate/up, 5 down + norm, 6 LM-head kernel alone, 7 top-k merge, 8 tree.
 * Errors: INVALID_ARG.
 */
int dart_set_profile_events(dart_handle* h, int stage, void* start_event, void* stop_event);

/*
 * Per-row log-softmax + top-k of caller-provided logits without any allocation (the paper has no
 * counterpart: this is the candidate selection of Algorithm 1 lines 6-8 at temperature 0, offered to
 * callers that cannot allocate device memory -- a process whose own pool already owns all of HBM, a
 * latency-critical loop where cudaMalloc's implicit synchronisation is not allowed, a plug-in without a
 * dart_handle to hold a workspace).  Needs no handle.
 *   logits      DEVICE f32 [rows, vocab], row-major            (in)
 *   out_ids     DEVICE i32 [rows, topk]   value desc, ties to the lower id   (out)
 *   out_slogit  DEVICE f32 [rows, topk]   log(softmax(logits)[id] + eps_logit) (out)
 * Limits: 1 <= rows <= 128 (more: DART_ERR_CAPACITY), 1 <= topk <= min(32, vocab).
 * Scratch: a fixed 1.6 MB array inside the library's device image, one per GPU, which every GPU that
 * loads the library holds until the process exits.  All calls on a GPU share it and it keeps the last
 * call's contents (every call overwrites what it reads, nothing needs clearing): calls that overlap on
 * the same GPU -- different streams or host threads -- race; serialise them.
 * The first call on each device (made with that device current) looks up the array's device address
 * (two host threads making it together both cache the same address, which is harmless);
 * make that first call before any CUDA stream capture.  Calls cudaMalloc/cudaFree never.
 * Asynchronous on `cuda_stream`.  Errors: INVALID_ARG, CAPACITY, UNSUPPORTED_ARCH (not sm_100),
 * CUDA (the cudaError_t is then returned by dart_last_cuda_error(NULL)).
 */
int dart_topk_rows_noalloc(const float* logits, int32_t rows, int32_t vocab, int32_t topk, float eps_logit,
                           int32_t* out_ids, float* out_slogit, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* DART_H_ */
