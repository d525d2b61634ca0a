// LM head with fused vocab-sharded log-softmax + per-position top-k
// (Section 3.2: one logit row per future position; Algorithm 1 lines 6-8; Appendix D s_logit).
//
// The LM head is 63 % of the step's bytes at the Qwen3-14B shape, so it is the kernel the roofline is
// quoted on.  Two kernels live here: lm_head_umma_kernel for up to 32 token rows and lm_head_dense_kernel for
// 33..128 (operands swapped), both with a TMA-fed shared-memory ring, tcgen05.mma and the logits in tensor memory.
// Complete logits never leave the SM: they are folded into a running (max, sum-exp) pair and an exact top-32
// list per token row.  A CTA writes (max, sum-exp, list) per token row; topk_merge_kernel (topk_merge.cu)
// combines the CTAs' results and emits the k best ids with s_logit = log(softmax + eps).
//
// With temperature > 0 the list is ordered by logit/T + Gumbel noise (Gumbel-top-k = sampling
// without replacement); the noise of token v in row (b, r) is word v&3 of
// Philox4x32-10(counter = (v>>2, r, b, step), key = seed): a lane folds four consecutive tokens per call.
#include <string.h>

#include "common.cuh"
#include "kernels.h"
#include "umma.cuh"
#include "select.cuh"

namespace dart {

__device__ __forceinline__ float gumbel_from_bits(uint32_t x) {
  // u = ((x >> 8) + 0.5) * 2^-24 in (0, 1); G = -log(-log u).  fp32 throughout (two fp64 logarithms per logit
  // were the LM head's largest cost at temperature > 0: 690 of 1330 us at 128 token rows).  Near u = 1 the
  // inner logarithm goes through log1p of the exact distance to 1, so the top bits of x keep their say.
  const uint32_t m = x >> 8;
  float t;
  if (m >= (1u << 23)) t = -log1pf(-(((float)((1u << 24) - m) - 0.5f) * (1.f / 16777216.f)));
  else t = -logf(((float)m + 0.5f) * (1.f / 16777216.f));
  return -logf(t);
}

// Insert (key, y, id) into the warp-resident list (lane j holds the j-th best; order: key desc, id asc).
__device__ __forceinline__ void list_insert(float& lk, float& ly, int& lid, float nk, float ny, int nid, int lane) {
  const bool before = (lk > nk) || (lk == nk && lid < nid);
  const int pos = __popc(__ballot_sync(0xffffffffu, before));
  const float pk = __shfl_up_sync(0xffffffffu, lk, 1), py = __shfl_up_sync(0xffffffffu, ly, 1);
  const int pid = __shfl_up_sync(0xffffffffu, lid, 1);
  if (lane == pos) { lk = nk; ly = ny; lid = nid; }
  else if (lane > pos) { lk = pk; ly = py; lid = pid; }
}

// Folds `nrows` (<= 128) complete logits of token row tk (srow[0 .. nrows), vocabulary ids id0 + index) into
// the CTA's running softmax statistics and its exact top list of that row (Algorithm 1 lines 6-8).  One warp.
__device__ __forceinline__ void fold_token(const LmParams& p, const float* srow, int nrows, int id0, int tk, int lane,
                                           float* st_key, float* st_y, int* st_id, float* st_ms) {
  float lk = st_key[tk * 32 + lane], ly = st_y[tk * 32 + lane];
  int lid = st_id[tk * 32 + lane];
  float m_run = st_ms[2 * tk], s_run = st_ms[2 * tk + 1];
  // lane owns the four consecutive vocabulary rows 4*lane .. 4*lane+3 of the 128: one Philox call covers them
  float yv[4], kv[4];
  float tmax = -INFINITY;
  uint4 rnd = make_uint4(0, 0, 0, 0);
  if (p.gumbel && 4 * lane < nrows)
    rnd = philox4x32_10(make_uint4((uint32_t)(id0 >> 2) + lane, (uint32_t)(tk % p.K), (uint32_t)(tk / p.K), p.step), p.seed_lo, p.seed_hi);
  const uint32_t rw[4] = {rnd.x, rnd.y, rnd.z, rnd.w};
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int idx = 4 * lane + q;
    const bool ok = idx < nrows;
    yv[q] = ok ? srow[idx] * p.inv_temp : -INFINITY;
    kv[q] = yv[q];
    if (p.gumbel && ok) kv[q] = yv[q] + gumbel_from_bits(rw[q]);
    tmax = fmaxf(tmax, yv[q]);
  }
  tmax = warp_max(tmax);
  const float m_new = fmaxf(m_run, tmax);
  float part = 0.f;
#pragma unroll
  for (int q = 0; q < 4; ++q) part += (4 * lane + q < nrows) ? expf(yv[q] - m_new) : 0.f;
  part = warp_sum(part);
  s_run = s_run * expf(m_run - m_new) + part;
  m_run = m_new;
  float thr = __shfl_sync(0xffffffffu, lk, p.topk - 1);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const bool ok = 4 * lane + q < nrows;
    unsigned mask = __ballot_sync(0xffffffffu, ok && kv[q] > thr);
    while (mask) {
      const int src = __ffs(mask) - 1;
      const float nk = __shfl_sync(0xffffffffu, kv[q], src), ny = __shfl_sync(0xffffffffu, yv[q], src);
      list_insert(lk, ly, lid, nk, ny, id0 + 4 * src + q, lane);
      thr = __shfl_sync(0xffffffffu, lk, p.topk - 1);
      mask &= mask - 1;
      mask &= __ballot_sync(0xffffffffu, ok && kv[q] > thr);
    }
  }
  st_key[tk * 32 + lane] = lk;
  st_y[tk * 32 + lane] = ly;
  st_id[tk * 32 + lane] = lid;
  if (lane == 0) { st_ms[2 * tk] = m_run; st_ms[2 * tk + 1] = s_run; }
}

// ------------------------------------------------------------------------------------------------------
// Up to 32 token rows: weights and activation slices arrive by TMA in a ring of
// shared-memory stages, tcgen05.mma multiplies them straight from there (M = 128 vocabulary rows, N = hi and
// lo token rows), the fp32 logits of a tile sit in tensor memory until four warps read them out and fold them.
//
// Work split: the flattened (128-row vocabulary tile, 64-k block) space is cut into gridDim.x equal ranges
// (one persistent CTA per SM), so every CTA streams the same number of bytes even though V / 128 is no
// multiple of the SM count.  A tile cut between CTAs belongs to the CTA that holds its first k-block: the
// others (for which it is the *first* thing they do) write their partial logits to a piece slot and raise a
// flag; the owner (for which it is the *last* thing it does) adds them in CTA order and folds.  Ownership
// is static, so the per-CTA statistics and lists - and with them every output bit - do not depend on timing.
// The owner's wait on the flags is bounded like every other wait here.
// ------------------------------------------------------------------------------------------------------
using namespace umma;

constexpr int kLmUmmaThreads = 512;   // producer, MMA issuer, TMEM owner, one idle warp; four read-out and eight more fold warps

template <int MP>
struct LmUmmaCfg {
  static constexpr int N = 2 * MP;
  static constexpr int XBytes = N * 64 * 2;
#ifndef LM_KS
#define LM_KS 2
#endif
  // A stage holds KS consecutive 64-k blocks of a vocabulary tile: KS weight boxes, then KS activation slices.  A
  // stage of the ring costs about the same ~690 cycles whatever it holds, and with one block (16 KB of weights) that
  // is 23 bytes per clock: just an SM's share of HBM.
  static constexpr int KS = LM_KS;
  static constexpr int StageBytes = KS * (128 * 64 * 2 + XBytes);
  static constexpr int TmemCols = 2 * N < 32 ? 32 : 2 * N;
  // epilogue shared memory: stage [MP][129] floats, lists 3 x [MP][32], statistics [MP][2], 1/rms [MP]
  static constexpr size_t EpiBytes = sizeof(float) * (MP * 129 + 3 * MP * 32 + 3 * MP);
  static constexpr int Stages = (MP == 8 ? 11 : 7) / KS + (KS > 1 && MP == 32 ? 1 : 0);
  static constexpr size_t SmemBytes = (size_t)Stages * StageBytes + 1024 + EpiBytes;
};

template <int MP>
__global__ void __launch_bounds__(kLmUmmaThreads, 1) lm_head_umma_kernel(const __grid_constant__ LmUmmaArgs a) {
  using C = LmUmmaCfg<MP>;
  constexpr int SROW = 129;
  const LmParams& p = a.p;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  float* stage = reinterpret_cast<float*>(ring + (size_t)C::Stages * C::StageBytes);   // [MP][SROW]
  float* st_key = stage + MP * SROW;         // [MP][32]
  float* st_y = st_key + MP * 32;
  int* st_id = reinterpret_cast<int*>(st_y + MP * 32);
  float* st_ms = reinterpret_cast<float*>(st_id + MP * 32);  // [MP][2]
  float* s_rstd = st_ms + 2 * MP;                            // [MP]
  __shared__ uint64_t full[C::Stages], empty[C::Stages], acc_full[2], acc_empty[2];
  __shared__ uint32_t tmem_base;
  __shared__ int abort_flag, s_bad;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
  const int c = blockIdx.x, G = gridDim.x;
  const int KB = a.KB;
  const long long u0 = ((long long)c * a.U) / G, u1 = ((long long)(c + 1) * a.U) / G;

  if (tid == 0) {
    for (int s = 0; s < C::Stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 128); }
    abort_flag = 0;
    s_bad = 0;
    fence_barrier_init();
    // this thread is the producer: the ring is filled with weights before anything else of the CTA's setup
    const int n = (int)(u1 - u0);
    const int pre = n < C::Stages ? n : C::Stages;
    const uint64_t wpol = l2_policy_evict_first();
    int tile = (int)(u0 / KB), kb = (int)(u0 % KB);
    for (int it = 0; it < pre; ++it) {
      mbar_expect_tx(&full[it], C::StageBytes);
#pragma unroll
      for (int q = 0; q < C::KS; ++q)
        tma_load_2d_hint(ring + (size_t)it * C::StageBytes + q * (128 * 64 * 2), &a.mapW, &full[it], (kb * C::KS + q) * 64, tile * 128, wpol);
      if (++kb == KB) { kb = 0; ++tile; }
    }
  }
  if (warp == 2) tmem_alloc(&tmem_base, C::TmemCols);
  for (int i = tid; i < MP * 32; i += kLmUmmaThreads) { st_key[i] = -INFINITY; st_y[i] = 0.f; st_id[i] = 0x7fffffff; }
  for (int i = tid; i < MP; i += kLmUmmaThreads) { st_ms[2 * i] = -INFINITY; st_ms[2 * i + 1] = 0.f; }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base;

  if (warp == 0 && lane == 0) {
    // ---- producer (the ring already holds the first weights): activations depend on the previous kernel
    const int n = (int)(u1 - u0);
    const int pre = n < C::Stages ? n : C::Stages;
    const uint64_t wpol = l2_policy_evict_first();
    int tile, kb;
    pdl_wait();
    tile = (int)(u0 / KB); kb = (int)(u0 % KB);
    for (int it = 0; it < pre; ++it) {
      uint8_t* xs = ring + (size_t)it * C::StageBytes + C::KS * (128 * 64 * 2);
#pragma unroll
      for (int q = 0; q < C::KS; ++q) tma_load_3d(xs + q * C::XBytes, &a.mapXhi, &full[it], (kb * C::KS + q) * 64, 0, 0);
      if (++kb == KB) { kb = 0; ++tile; }
    }
    int s = pre == C::Stages ? 0 : pre, ph = pre == C::Stages ? 1 : 0;
    for (int it = pre; it < n; ++it) {
      if (!mbar_wait(&empty[s], (ph - 1) & 1, &abort_flag)) break;
      uint8_t* st = ring + (size_t)s * C::StageBytes;
      mbar_expect_tx(&full[s], C::StageBytes);
#pragma unroll
      for (int q = 0; q < C::KS; ++q) {
        tma_load_2d_hint(st + q * (128 * 64 * 2), &a.mapW, &full[s], (kb * C::KS + q) * 64, tile * 128, wpol);
        tma_load_3d(st + C::KS * (128 * 64 * 2) + q * C::XBytes, &a.mapXhi, &full[s], (kb * C::KS + q) * 64, 0, 0);
      }
      if (++s == C::Stages) { s = 0; ++ph; }
      if (++kb == KB) { kb = 0; ++tile; }
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer
    constexpr uint32_t idesc = idesc_bf16(128, C::N);
    const int n = (int)(u1 - u0);
    int visit = -1, buf = 0, tile = -1;
    int t = (int)(u0 / KB), kb = (int)(u0 % KB), s = 0, ph = 0;
    bool ok = true;
    for (int it = 0; it < n && ok; ++it) {
      bool first = false;
      if (t != tile) {
        if (tile >= 0) mma_commit(&acc_full[buf]);
        tile = t;
        first = true;
        ++visit;
        buf = visit & 1;
        if (visit >= 2) {
          if (!mbar_wait(&acc_empty[buf], ((visit >> 1) - 1) & 1, &abort_flag)) { ok = false; break; }
          tc_fence_after();
        }
      }
      if (!mbar_wait(&full[s], ph & 1, &abort_flag)) { ok = false; break; }
      tc_fence_after();
      const uint32_t wa = smem_u32(ring + (size_t)s * C::StageBytes);
#pragma unroll
      for (int q = 0; q < C::KS; ++q) {
        const uint64_t ad = desc_sw128(wa + q * (128 * 64 * 2)), bd = desc_sw128(wa + C::KS * (128 * 64 * 2) + q * C::XBytes);
#pragma unroll
        for (int k = 0; k < 4; ++k) mma_f16(tmem + buf * C::N, ad + 2 * k, bd + 2 * k, idesc, (!first || q > 0 || k > 0) ? 1u : 0u);
      }
      mma_commit(&empty[s]);
      if (++s == C::Stages) { s = 0; ++ph; }
      if (++kb == KB) { kb = 0; ++t; }
    }
    if (ok && tile >= 0) mma_commit(&acc_full[buf]);
  } else if (warp >= 4) {
    // ---- read-out (warps 4-7: TMEM lane = vocabulary row of the tile) and fold (warps 4-15: one token row per warp
    // at a time).  A fold costs ~6000 cycles -- a CTA sees ~1000 vocabulary rows per token, so its running threshold
    // never gets selective and one value in seven is inserted -- and with 32 token rows on four warps that was 47000
    // cycles per tile against the 54000 the tile takes to stream: the MMA thread waited for a free accumulator a fifth
    // of the time (cycle counters).  On twelve warps it is three folds per tile and warp.
    // Every visit ends with the same two barriers for all twelve warps, and s_bad is only written between the second
    // of one visit and the first of the next, so a wait that ran out takes all of them out at the same place.
    const int fw = warp - 4;
    const bool reader = fw < 4;
    const int fi = reader ? fw + 8 : fw - 4;     // fold order: the warps that do not read out take the first rows
    const int wq = warp & 3, row = wq * 32 + lane, et = tid - 128;
    pdl_wait();
    if (reader) {
      // the final RMSNorm's per-token 1/rms comes from the previous kernel's sums of squares
      for (int i = et; i < MP; i += 128) {
        float ssq = 0.f;
        if (i < p.M)
          for (int tl = 0; tl < p.ss_tiles; ++tl) ssq += p.ss_in[(size_t)tl * p.ss_mp + i];
        s_rstd[i] = i < p.M ? 1.f / sqrtf(ssq / (float)p.Kd + p.rms_eps) : 0.f;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
    }
    int visit = 0;
    long long u = u0;
    while (u < u1) {
      const int tile = (int)(u / KB);
      const int ka = (int)(u - (long long)tile * KB);
      long long ue = (long long)(tile + 1) * KB;
      if (ue > u1) ue = u1;
      const bool owner = ka == 0, whole = owner && ue == (long long)(tile + 1) * KB;
      const int rows_here = min(128, p.V - tile * 128);
      if (reader) {
        const int buf = visit & 1;
        if (!mbar_wait_relaxed(&acc_full[buf], (visit >> 1) & 1, &abort_flag)) s_bad = 1;
        if (owner && !whole && et == 0) {
          // the rest of this tile comes from the next CTAs, for which it was the first thing to do
          for (int cc = c + 1; cc < G && ((long long)cc * a.U) / G < (long long)(tile + 1) * KB; ++cc) {
            int it = 0;
            while (*reinterpret_cast<volatile int*>(a.flags + cc) != a.tag && it < kSpinLimit) { __nanosleep(200); ++it; }
            if (it >= kSpinLimit) { s_bad = 1; abort_flag = 1; }
          }
          __threadfence();
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (!s_bad) {
          tc_fence_after();
          const uint32_t tbase = tmem + ((uint32_t)(wq * 32) << 16) + buf * C::N;
#pragma unroll 1
          for (int ch = 0; ch < MP / 8; ++ch) {
            uint32_t r[16];   // columns (2t, 2t+1) are token t's hi and lo parts
            tmem_ld16(tbase + ch * 16, r);
            tmem_ld_wait();
            float y[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) y[j] = __uint_as_float(r[2 * j]) + __uint_as_float(r[2 * j + 1]);
            if (ch == MP / 8 - 1) {  // the accumulator buffer is free once its last columns are in registers
              tc_fence_before();
              mbar_arrive(&acc_empty[buf]);
            }
            if (!owner) {
              float* dst = a.pieces + (((size_t)c * 128 + row) * MP + ch * 8);
              reinterpret_cast<float4*>(dst)[0] = make_float4(y[0], y[1], y[2], y[3]);
              reinterpret_cast<float4*>(dst)[1] = make_float4(y[4], y[5], y[6], y[7]);
              continue;
            }
            if (!whole) {
              for (int cc = c + 1; cc < G && ((long long)cc * a.U) / G < (long long)(tile + 1) * KB; ++cc) {
                const float* src = a.pieces + (((size_t)cc * 128 + row) * MP + ch * 8);
                const float4 q0 = __ldcg(reinterpret_cast<const float4*>(src)), q1 = __ldcg(reinterpret_cast<const float4*>(src) + 1);
                y[0] += q0.x; y[1] += q0.y; y[2] += q0.z; y[3] += q0.w;
                y[4] += q1.x; y[5] += q1.y; y[6] += q1.z; y[7] += q1.w;
              }
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int tok = ch * 8 + j;
              const float v = y[j] * s_rstd[tok];
              stage[tok * SROW + row] = v;
              if (p.logits_out != nullptr && tok < p.M && row < rows_here) p.logits_out[(size_t)tok * p.V + tile * 128 + row] = v;
            }
          }
          if (!owner) {
            // release the piece: every thread fences its part, then one thread raises this CTA's flag
            __threadfence();
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (et == 0) *reinterpret_cast<volatile int*>(a.flags + c) = a.tag;
          }
        }
      }
      asm volatile("bar.sync 2, 384;" ::: "memory");   // the tile's logits are staged (or a wait ran out)
      const bool bad = s_bad != 0;
      if (!bad && owner)
        for (int tk = fi; tk < p.M; tk += 12) fold_token(p, stage + tk * SROW, rows_here, tile * 128, tk, lane, st_key, st_y, st_id, st_ms);
      asm volatile("bar.sync 3, 384;" ::: "memory");   // the staging rows are free again
      if (bad) break;
      ++visit;
      u = ue;
    }
  }
  pdl_wait();
  pdl_trigger();
  __syncthreads();
  if (warp == 2) { tc_fence_after(); tmem_dealloc(tmem, C::TmemCols); }
  if (abort_flag || s_bad) {
    if (tid == 0) {
      atomicExch(a.status, DEV_TIMEOUT);
      for (int i = 0; i < 100; ++i) __nanosleep(1000);
    }
    __syncthreads();
  }
  for (int i = tid; i < MP * 32; i += kLmUmmaThreads) {
    const size_t o = (size_t)c * MP * 32 + i;
    p.part_key[o] = st_key[i];
    p.part_y[o] = st_y[i];
    p.part_id[o] = st_id[i];
  }
  for (int i = tid; i < MP * 2; i += kLmUmmaThreads) p.part_stats[(size_t)c * MP * 2 + i] = st_ms[i];
}

template <int MP>
static cudaError_t launch_lm_umma_t(const LmUmmaArgs& a, cudaStream_t st) {
  using C = LmUmmaCfg<MP>;
  const cudaError_t e = allow_dynamic_smem(reinterpret_cast<const void*>(lm_head_umma_kernel<MP>), C::SmemBytes);
  if (e != cudaSuccess) return e;
  return launch_pdl(lm_head_umma_kernel<MP>, dim3(a.p.grid), dim3(kLmUmmaThreads), C::SmemBytes, st, a);
}

// Units of work of a launch (what the grid is cut over): vocabulary tiles x ring stages per tile.
long long lm_head_units(int V, int Kd, bool dense) {
  const int kb = (Kd + 63) / 64;
  return dense ? (long long)((V + 255) / 256) * kb : (long long)((V + 127) / 128) * ((kb + LM_KS - 1) / LM_KS);
}

cudaError_t launch_lm_head_umma(const LmParams& pin, const CUtensorMap& mapW, const CUtensorMap& mapX,
                                float* pieces, int* flags, int tag, int* status, cudaStream_t st) {
  LmUmmaArgs a;
  memset(&a, 0, sizeof(a));
  a.p = pin;
  a.mapW = mapW; a.mapXhi = mapX;
  a.KB = ((pin.Kd + 63) / 64 + LM_KS - 1) / LM_KS;   // stages per vocabulary tile (a k tail reads as zeros)
  a.U = (long long)((pin.V + 127) / 128) * a.KB;
  a.pieces = pieces; a.flags = flags; a.tag = tag; a.status = status;
  const int MP = padded_tokens(pin.M);
  if (MP == 8) return launch_lm_umma_t<8>(a, st);
  if (MP == 32) return launch_lm_umma_t<32>(a, st);
  return cudaErrorInvalidValue;   // more token rows go to lm_head_dense_kernel
}

// ------------------------------------------------------------------------------------------------------
// LM head for 33..128 token rows: the operands swap sides.  With that many tokens the activation slice of a
// 64-k block (hi and lo rows of every token) is as large as the weight tile it meets, and re-reading it from L2
// for every 128 vocabulary rows is what bounds the kernel above (3 bytes through L2 per weight byte).  Here the
// token rows are the M side of tcgen05.mma (hi and lo as two MMAs into one accumulator) and 256 vocabulary rows
// its N side, so a stage carries 32 KB of activations for 32 KB of weights.  The accumulator row of a token
// is one TMEM lane, i.e. one read-out thread: that thread keeps the token's running (max, sum-exp) in registers
// and its best-`topk` candidates in a shared-memory row of its own (a heap rooted at the last-ranked entry; sorted
// once at the end), so the fold needs no cross-thread step at all.  Work split, ownership of tiles cut between CTAs, flags and
// bounded waits are those of lm_head_umma_kernel, with 256-row tiles.
// ------------------------------------------------------------------------------------------------------
// Two read-out threads per token row, one per half of a tile's 256 columns (warps 4-7 and 8-11), each with its own
// statistics and list: one warp per scheduler ran the fold at several cycles per instruction and was the longest
// part of the kernel; two halve that (fold on one warp set: 748 us).  The two sets of lists leave room for 160 KB of
// stages: three of weights and two of activations, in rings of their own (see the producer).
constexpr int kLmDenseWStages = 3, kLmDenseXStages = 2;
constexpr int kLmDenseThreads = 384;
constexpr int kLmDenseXBytes = 2 * 128 * 64 * 2;   // a stage of activations: hi tokens, lo tokens
constexpr int kLmDenseWBytes = 256 * 64 * 2;       // a stage of weights: 256 vocabulary rows
constexpr int kLmDenseRingBytes = kLmDenseXStages * kLmDenseXBytes + kLmDenseWStages * kLmDenseWBytes;
// lists: entry e of token row t of half h at [h][e][t] -- a thread's entries are 128 floats apart, so whichever
// entries the lanes of a warp touch, they touch 32 different banks
constexpr size_t kLmDenseSmem = (size_t)kLmDenseRingBytes + 1024 + 2 * 2 * 32 * 128 * 4 + 2 * 128 * 4;

// (key, id) a precedes (key, id) b in the candidate order: larger key first, then smaller id
__device__ __forceinline__ bool cand_before(float ka, int ia, float kb, int ib) { return ka > kb || (ka == kb && ia < ib); }

__global__ void __launch_bounds__(kLmDenseThreads, 1) lm_head_dense_kernel(const __grid_constant__ LmUmmaArgs a) {
  const LmParams& p = a.p;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* ring_x = ring;                                                  // [2][hi | lo]
  uint8_t* ring_w = ring + kLmDenseXStages * kLmDenseXBytes;               // [3]
  float* l_key = reinterpret_cast<float*>(ring + kLmDenseRingBytes);       // [2 halves][32][128]
  int* l_id = reinterpret_cast<int*>(l_key + 2 * 32 * 128);                // [2 halves][32][128]
  volatile float* l_thr = reinterpret_cast<volatile float*>(l_id + 2 * 32 * 128);  // [2 halves][128] published thresholds
  __shared__ uint64_t full_w[kLmDenseWStages], empty_w[kLmDenseWStages], full_x[kLmDenseXStages], empty_x[kLmDenseXStages];
  __shared__ uint64_t acc_full[2], acc_empty[2];
  __shared__ uint32_t tmem_base;
  __shared__ int abort_flag, s_bad;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
  const int c = blockIdx.x, G = gridDim.x;
  const int KB = a.KB;
  const long long u0 = ((long long)c * a.U) / G, u1 = ((long long)(c + 1) * a.U) / G;
  constexpr int kXBytes = 128 * 64 * 2;

  if (tid == 0) {
    for (int s = 0; s < kLmDenseWStages; ++s) { mbar_init(&full_w[s], 1); mbar_init(&empty_w[s], 1); }
    for (int s = 0; s < kLmDenseXStages; ++s) { mbar_init(&full_x[s], 1); mbar_init(&empty_x[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 256); }
    abort_flag = 0;
    s_bad = 0;
    fence_barrier_init();
    // the producer fills the weight stages before anything else of the CTA's setup
    const int n = (int)(u1 - u0);
    const int pre = n < kLmDenseWStages ? n : kLmDenseWStages;
    const uint64_t wpol = l2_policy_evict_first();
    int tile = (int)(u0 / KB), kb = (int)(u0 % KB);
    for (int it = 0; it < pre; ++it) {
      mbar_expect_tx(&full_w[it], kLmDenseWBytes);
      tma_load_2d_hint(ring_w + (size_t)it * kLmDenseWBytes, &a.mapW, &full_w[it], kb * 64, tile * 256, wpol);
      if (++kb == KB) { kb = 0; ++tile; }
    }
  }
  if (warp == 2) tmem_alloc(&tmem_base, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base;

  if (warp == 0 && lane == 0) {
    // ---- producer.  Weights and activations have rings of their own: three weight stages, so that a refill has two
    // stages' worth of MMAs to arrive from HBM, and two for the activation slices, which come from L2.  Unit it reads
    // weight stage it mod 3 and activation stage it mod 2.  Cycle counters at 128 token rows: the MMA thread spends
    // ~960 cycles per stage issuing (the eight MMAs of a stage take 1024 on the tensor pipe) and waits 270 for weights
    // and 620 for activations (985 with two stages of both).  The launch did not get shorter for it: it runs under the
    // power cap (600 000 cycles in 368 us on the global timer -- 1.6 GHz -- in a run of three steps, fewer MHz still
    // in a long one), where fewer stalled cycles buy a lower clock.
    const int n = (int)(u1 - u0);
    const uint64_t wpol = l2_policy_evict_first();
    pdl_wait();
    int xkb = (int)(u0 % KB);                                  // k-block of the next activation slice
    int wt = (int)(u0 / KB), wkb = (int)(u0 % KB);             // tile and k-block of the next weight stage
    auto load_x = [&](int s) {
      uint8_t* st = ring_x + (size_t)s * kLmDenseXBytes;
      mbar_expect_tx(&full_x[s], kLmDenseXBytes);
      tma_load_2d(st, &a.mapXhi, &full_x[s], xkb * 64, 0);
      tma_load_2d(st + kXBytes, &a.mapXlo, &full_x[s], xkb * 64, 0);
      if (++xkb == KB) xkb = 0;
    };
    for (int it = 0; it < n && it < kLmDenseXStages; ++it) load_x(it);
    for (int it = 0; it < n && it < kLmDenseWStages; ++it)     // already requested above
      if (++wkb == KB) { wkb = 0; ++wt; }
    // from unit 2 on, both refills wait for the MMAs of unit it - 2: weights of unit it + 1, activations of unit it
    int ws = 0, wph = 0;
    for (int it = 2; it < n; ++it) {
      if (it + 1 < n) {
        if (!mbar_wait(&empty_w[ws], wph & 1, &abort_flag)) break;
        mbar_expect_tx(&full_w[ws], kLmDenseWBytes);
        tma_load_2d_hint(ring_w + (size_t)ws * kLmDenseWBytes, &a.mapW, &full_w[ws], wkb * 64, wt * 256, wpol);
        if (++wkb == KB) { wkb = 0; ++wt; }
        if (++ws == kLmDenseWStages) { ws = 0; ++wph; }
      }
      if (!mbar_wait(&empty_x[it & 1], ((it >> 1) - 1) & 1, &abort_flag)) break;
      load_x(it & 1);
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer: D[token, vocabulary row] += (X_hi + X_lo)[token, k] * W[vocabulary row, k]
    constexpr uint32_t idesc = idesc_bf16(128, 256);
    const int n = (int)(u1 - u0);
    int visit = -1, buf = 0, tile = -1;
    int t = (int)(u0 / KB), kb = (int)(u0 % KB), ws = 0, wph = 0;
    bool ok = true;
    for (int it = 0; it < n && ok; ++it) {
      bool first = false;
      if (t != tile) {
        if (tile >= 0) mma_commit(&acc_full[buf]);
        tile = t;
        first = true;
        ++visit;
        buf = visit & 1;
        if (visit >= 2) {
          if (!mbar_wait(&acc_empty[buf], ((visit >> 1) - 1) & 1, &abort_flag)) { ok = false; break; }
          tc_fence_after();
        }
      }
      const int xs = it & 1;
      if (!mbar_wait(&full_w[ws], wph & 1, &abort_flag)) { ok = false; break; }
      if (!mbar_wait(&full_x[xs], (it >> 1) & 1, &abort_flag)) { ok = false; break; }
      tc_fence_after();
      const uint32_t xa = smem_u32(ring_x + (size_t)xs * kLmDenseXBytes);
      const uint64_t hd = desc_sw128(xa), ld = desc_sw128(xa + kXBytes), wd = desc_sw128(smem_u32(ring_w + (size_t)ws * kLmDenseWBytes));
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        mma_f16(tmem + buf * 256, hd + 2 * k, wd + 2 * k, idesc, (!first || k > 0) ? 1u : 0u);
        mma_f16(tmem + buf * 256, ld + 2 * k, wd + 2 * k, idesc, 1u);
      }
      mma_commit(&empty_w[ws]);
      mma_commit(&empty_x[xs]);
      if (++ws == kLmDenseWStages) { ws = 0; ++wph; }
      if (++kb == KB) { kb = 0; ++t; }
    }
    if (ok && tile >= 0) mma_commit(&acc_full[buf]);
  } else if (warp >= 4) {
    // ---- read-out and fold: TMEM lane = token row; this thread owns one half of the columns of the token's row of
    // every tile, with statistics and a list of its own (the two halves are merged at the end)
    const int wq = warp & 3, half = (warp - 4) >> 2, tok = wq * 32 + lane, et = tid - 128;
    const bool live = tok < p.M;
    float* my_key = l_key + half * 32 * 128 + tok;      // entry e at my_key[(e * 128) * 128]
    int* my_id = l_id + half * 32 * 128 + tok;
    pdl_wait();
    float rstd = 0.f;
    if (live) {  // the final RMSNorm's 1/rms from the previous kernel's sums of squares (same order everywhere)
      float ssq = 0.f;
      for (int tl = 0; tl < p.ss_tiles; ++tl) ssq += p.ss_in[(size_t)tl * p.ss_mp + tok];
      rstd = 1.f / sqrtf(ssq / (float)p.Kd + p.rms_eps);
    }
    float m_run = -INFINITY, s_run = 0.f;
    // The token's candidates: a binary heap in this thread's shared-memory row, its root the last-ranked entry kept,
    // i.e. the exact threshold a new logit has to precede.  An insertion is a walk of at most five levels, so a
    // warp whose rows insert at different moments loses little (replace-the-worst rescanned all `topk` entries
    // whenever any row inserted; append-and-compact paid ~4000 instructions per compaction).
    // Each half publishes the key of its heap's root once it holds `topk` entries: the other half of the same row
    // may skip whatever is below it too (topk entries of the row's union are at least that large), which takes away
    // close to half of the insertions.  A stale value only prunes less; the merged list does not depend on timing.
    l_thr[half * 128 + tok] = -INFINITY;
    int n_list = 0;
    const int topk = p.topk;
    // A bound shared by all CTAs.  A CTA sees ~1000 vocabulary rows of a token, so its own thresholds let one logit
    // in five through, and the insertions (~2300 cycles per warp round: cycle counters) were 4/5 of this role's time.
    // Every (CTA, half) publishes the largest key it has met so far for the token -- at temperature > 0 a lower
    // bound of it -- into slot (2 c + half) mod (topk + 7) of the token's row of `bound` (atomic max; the launch's
    // tag in the upper word makes older launches' values invalid without a reset).  The slots hold keys of distinct
    // vocabulary rows, so the topk-th largest slot -- the 8th smallest -- is at most the topk-th largest key of the
    // whole vocabulary: whatever is below it cannot be in the result.  After one 16-logit chunk per thread that is
    // already the 99th percentile.  A stale or missing value only prunes less: which candidates a CTA keeps depends
    // on timing, the merged top list does not.
    const int n_slots = topk + 7;
    unsigned long long* g_row = a.bound + (size_t)tok * kLmBoundSlots;
    const int g_slot = (2 * c + half) % n_slots;
    const unsigned long long g_tag = (unsigned long long)(uint32_t)a.tag << 32;
    float tau = -INFINITY, pub = -INFINITY;
    int n_own = 0;                               // chunks of owned tiles folded so far
    auto refresh_tau = [&]() {
      float s8[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) s8[q] = INFINITY;
      for (int i = 0; i < n_slots; ++i) {
        const unsigned long long w = __ldcg(g_row + i);
        float v = (w >> 32) == (g_tag >> 32) ? float_unorder((uint32_t)w) : -INFINITY;
#pragma unroll
        for (int q = 0; q < 8; ++q) { const float lo = fminf(s8[q], v); v = fmaxf(s8[q], v); s8[q] = lo; }
      }
      tau = s8[7];
    };
    auto worse = [&](int x, int y) { return cand_before(my_key[(y) * 128], my_id[(y) * 128], my_key[(x) * 128], my_id[(x) * 128]); };   // entry x ranks after entry y
    auto heap_insert = [&](float ke, int ie) {
      if (n_list < topk) {                       // grow: the new leaf rises while it ranks after its parent
        int i = n_list++;
        while (i > 0) {
          const int up = (i - 1) >> 1;
          if (!cand_before(my_key[(up) * 128], my_id[(up) * 128], ke, ie)) break;          // the parent does not rank before it: stop
          my_key[(i) * 128] = my_key[(up) * 128]; my_id[(i) * 128] = my_id[(up) * 128];
          i = up;
        }
        my_key[(i) * 128] = ke; my_id[(i) * 128] = ie;
      } else if (cand_before(ke, ie, my_key[(0) * 128], my_id[(0) * 128])) {               // replace the root, sink it
        int i = 0;
        for (;;) {
          int ch = 2 * i + 1;
          if (ch >= topk) break;
          if (ch + 1 < topk && worse(ch + 1, ch)) ++ch;                    // the later-ranked child
          if (!cand_before(ke, ie, my_key[(ch) * 128], my_id[(ch) * 128])) break;          // the new entry ranks after both children
          my_key[(i) * 128] = my_key[(ch) * 128]; my_id[(i) * 128] = my_id[(ch) * 128];
          i = ch;
        }
        my_key[(i) * 128] = ke; my_id[(i) * 128] = ie;
      }
    };
    int visit = 0;
    long long u = u0;
    while (u < u1) {
      const int tile = (int)(u / KB);
      const int ka = (int)(u - (long long)tile * KB);
      long long ue = (long long)(tile + 1) * KB;
      if (ue > u1) ue = u1;
      const bool owner = ka == 0, whole = owner && ue == (long long)(tile + 1) * KB;
      const int buf = visit & 1;
      if (!mbar_wait_relaxed(&acc_full[buf], (visit >> 1) & 1, &abort_flag)) s_bad = 1;
      if (owner && !whole && et == 0) {
        for (int cc = c + 1; cc < G && ((long long)cc * a.U) / G < (long long)(tile + 1) * KB; ++cc) {
          int it = 0;
          while (*reinterpret_cast<volatile int*>(a.flags + cc) != a.tag && it < kSpinLimit) { __nanosleep(200); ++it; }
          if (it >= kSpinLimit) { s_bad = 1; abort_flag = 1; }
        }
        __threadfence();
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (s_bad) break;
      tc_fence_after();
      const uint32_t tbase = tmem + ((uint32_t)(wq * 32) << 16) + buf * 256;
#pragma unroll 1
      for (int cb = half * 128; cb < half * 128 + 128; cb += 16) {
        uint32_t r[16];
        tmem_ld16(tbase + cb, r);
        tmem_ld_wait();
        if (cb == half * 128 + 112) {  // the accumulator buffer is free once both halves' last columns are in registers
          tc_fence_before();
          mbar_arrive(&acc_empty[buf]);
        }
        float y[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) y[j] = __uint_as_float(r[j]);
        if (!owner) {
          float4* dst = reinterpret_cast<float4*>(a.pieces + (((size_t)c * 128 + tok) * 256 + cb));
#pragma unroll
          for (int j = 0; j < 4; ++j) dst[j] = make_float4(y[4 * j], y[4 * j + 1], y[4 * j + 2], y[4 * j + 3]);
          continue;
        }
        if (!whole) {
          for (int cc = c + 1; cc < G && ((long long)cc * a.U) / G < (long long)(tile + 1) * KB; ++cc) {
            const float4* src = reinterpret_cast<const float4*>(a.pieces + (((size_t)cc * 128 + tok) * 256 + cb));
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float4 q = __ldcg(src + j);
              y[4 * j] += q.x; y[4 * j + 1] += q.y; y[4 * j + 2] += q.z; y[4 * j + 3] += q.w;
            }
          }
        }
        const int v0 = tile * 256 + cb;             // vocabulary id of column 0 of this chunk (a multiple of 16)
        if (v0 >= p.V) continue;                    // the same for every lane: what follows is warp-collective
#pragma unroll
        for (int j = 0; j < 16; ++j) y[j] *= rstd;
        if (live && p.logits_out != nullptr) {
          float4* lo = reinterpret_cast<float4*>(p.logits_out + (size_t)tok * p.V + v0);
#pragma unroll
          for (int j = 0; j < 4; ++j) lo[j] = make_float4(y[4 * j], y[4 * j + 1], y[4 * j + 2], y[4 * j + 3]);
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) y[j] *= p.inv_temp;
        {  // running log-sum-exp of this token row, one chunk at a time (independent exponentials overlap)
          float cm = y[0];
#pragma unroll
          for (int j = 1; j < 16; ++j) cm = fmaxf(cm, y[j]);
          if (cm > m_run) { s_run *= __expf(m_run - cm); m_run = cm; }
          float e4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int j = 0; j < 16; ++j) e4[j & 3] += __expf(y[j] - m_run);   // ex2.approx: ~2e-6 relative, far inside s_logit's tolerance
          s_run += (e4[0] + e4[1]) + (e4[2] + e4[3]);
        }
        // which of the 16 logits may precede the threshold (the heap's root once `topk` are kept).  At temperature
        // > 0 the key is y + G(u): a fast evaluation of G decides with a margin 10x its error bound (u in
        // [2^-14, 1 - 2^-8]: |error| < 1.2e-4; other u always pass); the exact fp32 G is computed for those only.
        const bool full = n_list == topk;
        const float o_key = fmaxf(l_thr[(half ^ 1) * 128 + tok], tau);   // the other half's threshold and the shared bound (or -inf)
        const float t_key = full ? my_key[(0) * 128] : -INFINITY;
        const int t_id = full ? my_id[(0) * 128] : 0x7fffffff;
        if (full) l_thr[half * 128 + tok] = t_key;
        uint32_t may = 0u;
        uint32_t bits[16];
        float kmax = -INFINITY;                  // a lower bound of the chunk's largest key
        if (p.gumbel) {
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            const uint4 rnd = philox4x32_10(make_uint4((uint32_t)((v0 >> 2) + q4), (uint32_t)(tok % p.K), (uint32_t)(tok / p.K), p.step), p.seed_lo, p.seed_hi);
            bits[4 * q4] = rnd.x; bits[4 * q4 + 1] = rnd.y; bits[4 * q4 + 2] = rnd.z; bits[4 * q4 + 3] = rnd.w;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const uint32_t m = bits[4 * q4 + q] >> 8;
              const float gq = -__logf(-__logf(((float)m + 0.5f) * (1.f / 16777216.f)));
              const bool safe = m >= 1024u && m <= (1u << 24) - 65536u;
              const float kq = y[4 * q4 + q] + gq + 1e-3f;
              if (safe) kmax = fmaxf(kmax, kq - 2e-3f);
              if ((!full || !safe || kq >= t_key) && (!safe || kq >= o_key)) may |= 1u << (4 * q4 + q);
            }
          }
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            bits[j] = 0u;
            kmax = fmaxf(kmax, y[j]);
            if ((!full || cand_before(y[j], v0 + j, t_key, t_id)) && y[j] >= o_key) may |= 1u << j;
          }
        }
        if (!live) may = 0u;
        if (live && kmax > pub) {
          atomicMax(g_row + g_slot, g_tag | float_order(kmax));
          pub = kmax;
        }
#pragma unroll 1
        while (may != 0u) {                      // one candidate per round; rows of a warp go through their rounds together
          const int j = __ffs(may) - 1;
          may &= may - 1u;
          float yj = y[0];
          uint32_t bj = bits[0];
#pragma unroll
          for (int q = 1; q < 16; ++q) { yj = q == j ? y[q] : yj; bj = q == j ? bits[q] : bj; }
          const float kj = p.gumbel ? yj + gumbel_from_bits(bj) : yj;
          if (kj >= o_key) heap_insert(kj, v0 + j);
        }
        // the shared bound is read again after 1, 2, 4, 8 chunks and then once per tile half
        ++n_own;
        if (live && (n_own <= 8 ? (n_own & (n_own - 1)) == 0 : (n_own & 7) == 0)) refresh_tau();
      }
      if (!owner) {
        __threadfence();
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (et == 0) *reinterpret_cast<volatile int*>(a.flags + c) = a.tag;
      }
      ++visit;
      u = ue;
    }
    // ---- this token's list, sorted (key desc, id asc), and its statistics
    // ---- the second half's statistics and list join the first half's (the ring is free by now: scratch)
    float* x_m = reinterpret_cast<float*>(ring);
    float* x_s = x_m + 128;
    int* x_n = reinterpret_cast<int*>(x_s + 128);
    if (half == 1) { x_m[tok] = m_run; x_s[tok] = s_run; x_n[tok] = n_list; }
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (half == 0) {
      const float m1 = x_m[tok], s1 = x_s[tok];
      if (m1 != -INFINITY) {
        const float mn = fmaxf(m_run, m1);
        s_run = (m_run == -INFINITY ? 0.f : s_run * expf(m_run - mn)) + s1 * expf(m1 - mn);
        m_run = mn;
      }
      const float* k1 = l_key + 32 * 128 + tok;
      const int* i1 = l_id + 32 * 128 + tok;
      const int n1 = x_n[tok];
      for (int e1 = 0; e1 < n1; ++e1) heap_insert(k1[e1 * 128], i1[e1 * 128]);
    }
    if (live && half == 0) {
      for (int i = 1; i < n_list; ++i) {            // insertion sort of at most 32 entries
        const float ki = my_key[(i) * 128]; const int ii = my_id[(i) * 128];
        int j = i - 1;
        while (j >= 0 && cand_before(ki, ii, my_key[(j) * 128], my_id[(j) * 128])) { my_key[(j + 1) * 128] = my_key[(j) * 128]; my_id[(j + 1) * 128] = my_id[(j) * 128]; --j; }
        my_key[(j + 1) * 128] = ki; my_id[(j + 1) * 128] = ii;
      }
      const size_t o = ((size_t)c * 128 + tok) * 32;
      for (int e = 0; e < 32; ++e) {
        const bool have = e < n_list;
        const float key = have ? my_key[(e) * 128] : -INFINITY;
        const int id = have ? my_id[(e) * 128] : 0x7fffffff;
        float yv = key;                                   // the un-perturbed logit / T of the entry
        if (have && p.gumbel) {
          const uint4 rnd = philox4x32_10(make_uint4((uint32_t)id >> 2, (uint32_t)(tok % p.K), (uint32_t)(tok / p.K), p.step), p.seed_lo, p.seed_hi);
          const uint32_t wsel = (id & 3) == 0 ? rnd.x : ((id & 3) == 1 ? rnd.y : ((id & 3) == 2 ? rnd.z : rnd.w));
          yv = key - gumbel_from_bits(wsel);
        }
        p.part_key[o + e] = key;
        p.part_y[o + e] = have ? yv : 0.f;
        p.part_id[o + e] = id;
      }
      p.part_stats[((size_t)c * 128 + tok) * 2] = m_run;
      p.part_stats[((size_t)c * 128 + tok) * 2 + 1] = s_run;
    }
  }
  pdl_wait();
  pdl_trigger();
  __syncthreads();
  if (warp == 2) { tc_fence_after(); tmem_dealloc(tmem, 512); }
  if ((abort_flag || s_bad) && tid == 0) {
    atomicExch(a.status, DEV_TIMEOUT);
    for (int i = 0; i < 100; ++i) __nanosleep(1000);
  }
  // token rows past M leave empty lists (the merge reads MP = 128 rows per CTA)
  for (int i = tid; i < (128 - p.M) * 32; i += kLmDenseThreads) {
    const size_t o = ((size_t)c * 128 + p.M) * 32 + i;
    p.part_key[o] = -INFINITY; p.part_y[o] = 0.f; p.part_id[o] = 0x7fffffff;
  }
  for (int i = tid; i < (128 - p.M) * 2; i += kLmDenseThreads) p.part_stats[((size_t)c * 128 + p.M) * 2 + i] = (i & 1) ? 0.f : -INFINITY;
}

cudaError_t launch_lm_head_dense(const LmParams& pin, const CUtensorMap& mapW256, const CUtensorMap& mapXhi, const CUtensorMap& mapXlo,
                                 float* pieces, int* flags, int tag, int* status, unsigned long long* bound, cudaStream_t st) {
  LmUmmaArgs a;
  memset(&a, 0, sizeof(a));
  a.p = pin;
  a.bound = bound;
  a.mapW = mapW256; a.mapXhi = mapXhi; a.mapXlo = mapXlo;
  a.KB = (pin.Kd + 63) / 64;
  a.U = (long long)((pin.V + 255) / 256) * a.KB;
  a.pieces = pieces; a.flags = flags; a.tag = tag; a.status = status;
  const cudaError_t e = allow_dynamic_smem(reinterpret_cast<const void*>(lm_head_dense_kernel), kLmDenseSmem);
  if (e != cudaSuccess) return e;
  return launch_pdl(lm_head_dense_kernel, dim3(a.p.grid), dim3(kLmDenseThreads), kLmDenseSmem, st, a);
}

}  // namespace dart
