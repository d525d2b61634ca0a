// LM head with fused vocab-sharded log-softmax + per-position top-k
// (Section 3.2: one logit row per future position; Algorithm 1 lines 6-8; Appendix D s_logit).
//
// The LM head is 63 % of the step's bytes at the Qwen3-14B shape, so it is the kernel the
// roofline is quoted on.  Each CTA owns a contiguous range of 16-row vocab tiles, balanced to
// within one tile, and streams them with the shared core of stream_core.cuh (16 warps interleave
// the k-steps of a tile, 2 CTAs per SM; the partial tiles are summed through shared memory).  Complete logits never leave the SM: every 128 vocab rows a warp per
// token row folds them into a running (max, sum-exp) pair and an exact top-32 list held one
// entry per lane.  The CTA writes (max, sum-exp, list) per token row; topk_merge_kernel
// (topk_merge.cu) combines the CTAs' results and emits the k best ids with s_logit = log(softmax + eps).
//
// With temperature > 0 the list is ordered by logit/T + Gumbel noise (Gumbel-top-k = sampling
// without replacement); the noise of token v in row (b, r) is word v&3 of
// Philox4x32-10(counter = (v>>2, r, b, step), key = seed).
#include <string.h>

#include "common.cuh"
#include "kernels.h"
#include "stream_core.cuh"

namespace dart {

__device__ __forceinline__ float gumbel_from_bits(uint32_t x) {
  // u = ((x >> 8) + 0.5) * 2^-24 in (0,1); fp64 so that u never rounds to 1
  const double u = ((double)(x >> 8) + 0.5) * (1.0 / 16777216.0);
  return (float)(-log(-log(u)));
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

// Epilogue functor of the streaming core: complete logits of a 16-row vocab tile -> stage; every 128
// staged vocab rows a warp per token row folds them into the running softmax statistics and top list.
template <int NT, int NW>
struct LmEpi {
  static constexpr int MP = 8 * NT;
  static constexpr int SROW = 128 + 1;  // stage row stride (floats)
  const LmParams& p;
  const float* red;
  float* stage;   // [MP][SROW]
  float* st_key; float* st_y; int* st_id; float* st_ms; float* s_rstd;
  int mt0;

  // the final RMSNorm's per-token 1/rms comes from the previous kernel's sums of squares
  __device__ __forceinline__ void after_wait() {
    for (int i = threadIdx.x; i < MP; i += NW * 32) {
      float ssq = 0.f;  // the activations are x * gain; their 1/rms multiplies the logits (same fixed order everywhere)
      if (i < p.M)
        for (int tl = 0; tl < p.ss_tiles; ++tl) ssq += p.ss_in[(size_t)tl * p.ss_mp + i];
      s_rstd[i] = i < p.M ? 1.f / sqrtf(ssq / (float)p.Kd + p.rms_eps) : 0.f;
    }
    __syncthreads();
  }

  __device__ __forceinline__ void mtile_done(int mt, int buf, bool last) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slot = (mt - mt0) & 7;
    for (int e = tid; e < 16 * MP; e += NW * 32) {
      const int row = e / MP, tok = e % MP;
      const float v = red_sum<NW, MP>(red, buf, row, tok) * s_rstd[tok];
      stage[tok * SROW + slot * 16 + row] = v;
      if (p.logits_out != nullptr && tok < p.M) p.logits_out[(size_t)tok * p.V + mt * 16 + row] = v;
    }
    if (slot == 7 || last) {
      __syncthreads();
      const int nrows = (slot + 1) * 16;
      const int id0 = (mt - slot) * 16;
      for (int tk = warp; tk < p.M; tk += NW) {
        float lk = st_key[tk * 32 + lane], ly = st_y[tk * 32 + lane];
        int lid = st_id[tk * 32 + lane];
        float m_run = st_ms[2 * tk], s_run = st_ms[2 * tk + 1];
        float yv[4], kv[4];
        float tmax = -INFINITY;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int idx = lane + 32 * q;
          const bool ok = idx < nrows;
          yv[q] = ok ? stage[tk * SROW + idx] * p.inv_temp : -INFINITY;
          kv[q] = yv[q];
          if (p.gumbel && ok) {
            const uint32_t v = (uint32_t)(id0 + idx);
            const uint4 rnd = philox4x32_10(make_uint4(v >> 2, (uint32_t)(tk % p.K), (uint32_t)(tk / p.K), p.step),
                                            p.seed_lo, p.seed_hi);
            const uint32_t wsel = (v & 3) == 0 ? rnd.x : ((v & 3) == 1 ? rnd.y : ((v & 3) == 2 ? rnd.z : rnd.w));
            kv[q] = yv[q] + gumbel_from_bits(wsel);
          }
          tmax = fmaxf(tmax, yv[q]);
        }
        tmax = warp_max(tmax);
        const float m_new = fmaxf(m_run, tmax);
        float part = 0.f;
#pragma unroll
        for (int q = 0; q < 4; ++q) part += (lane + 32 * q < nrows) ? expf(yv[q] - m_new) : 0.f;
        part = warp_sum(part);
        s_run = s_run * expf(m_run - m_new) + part;
        m_run = m_new;
        float thr = __shfl_sync(0xffffffffu, lk, p.topk - 1);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const bool ok = lane + 32 * q < nrows;
          unsigned mask = __ballot_sync(0xffffffffu, ok && kv[q] > thr);
          while (mask) {
            const int src = __ffs(mask) - 1;
            const float nk = __shfl_sync(0xffffffffu, kv[q], src), ny = __shfl_sync(0xffffffffu, yv[q], src);
            list_insert(lk, ly, lid, nk, ny, id0 + src + 32 * q, lane);
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
    }
  }
};

// FULL: Kd is a multiple of 64*NW and all rows/tokens are in range, so the streaming loop carries no
// bounds predicates at all.
template <int NT, int PF, int NW, bool FULL>
__global__ void __launch_bounds__(NW * 32, (NT == 1 ? 2 : 1)) lm_head_kernel(const __grid_constant__ LmParams p) {
  constexpr int MP = 8 * NT;
  constexpr int RB = (NT <= 4) ? 2 : 1;      // reduce buffers
  constexpr int SROW = 128 + 1;
  extern __shared__ __align__(16) float sm[];
  float* red = sm;                           // [RB][NW][16][MP]
  float* stage = red + RB * NW * 16 * MP;    // [MP][SROW]
  float* st_key = stage + MP * SROW;         // [MP][32]
  float* st_y = st_key + MP * 32;
  int* st_id = reinterpret_cast<int*>(st_y + MP * 32);
  float* st_ms = reinterpret_cast<float*>(st_id + MP * 32);  // [MP][2]
  float* s_rstd = st_ms + 2 * MP;                            // [MP] 1/rms of the final RMSNorm per token row

  const int c = blockIdx.x, G = gridDim.x, tid = threadIdx.x;
  const int n_mt = p.V >> 4;
  const int mt0 = (int)(((long long)c * n_mt) / G), mt1 = (int)(((long long)(c + 1) * n_mt) / G);

  for (int i = tid; i < MP * 32; i += NW * 32) { st_key[i] = -INFINITY; st_y[i] = 0.f; st_id[i] = 0x7fffffff; }
  for (int i = tid; i < MP; i += NW * 32) {
    st_ms[2 * i] = -INFINITY;
    st_ms[2 * i + 1] = 0.f;
  }
  __syncthreads();

  if (mt1 > mt0) {
    LmEpi<NT, NW> epi{p, red, stage, st_key, st_y, st_id, st_ms, s_rstd, mt0};
    stream_units<NT, true, PF, NW, RB, FULL>(p.s, (long long)mt0 * p.s.KR, (long long)mt1 * p.s.KR, red, epi);
  } else {
    pdl_wait();
  }
  pdl_trigger();
  __syncthreads();
  for (int i = tid; i < MP * 32; i += NW * 32) {
    const size_t o = (size_t)c * MP * 32 + i;
    p.part_key[o] = st_key[i];
    p.part_y[o] = st_y[i];
    p.part_id[o] = st_id[i];
  }
  for (int i = tid; i < MP * 2; i += NW * 32) p.part_stats[(size_t)c * MP * 2 + i] = st_ms[i];
}

template <int NT, int NW>
static size_t lm_smem_bytes() {
  constexpr int MP = 8 * NT, RB = (NT <= 4) ? 2 : 1;
  return sizeof(float) * ((size_t)RB * NW * 16 * MP + (size_t)MP * 129 + 3 * (size_t)MP * 32 + 3 * (size_t)MP);
}

template <int NT, int PF, int NW, bool FULL>
static cudaError_t launch_lm_t(LmParams& p, cudaStream_t st) {
  const size_t smem = lm_smem_bytes<NT, NW>();
  p.s.KR = (p.s.SK + NW - 1) / NW;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(lm_head_kernel<NT, PF, NW, FULL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  return launch_pdl(lm_head_kernel<NT, PF, NW, FULL>, dim3(p.grid), dim3(NW * 32), smem, st, p);
}

cudaError_t launch_lm_head(const LmParams& pin, cudaStream_t st) {
  LmParams p = pin;
  const int MP = padded_tokens(p.M);
  if (p.x_lo == nullptr) return cudaErrorInvalidValue;  // the LM head always takes hi + lo activations
  memset(&p.s, 0, sizeof(p.s));
  for (int i = 0; i < 6; ++i) p.s.seg[i] = GemmSeg{p.W, p.V, 0, p.Kd, 0};
  p.s.nseg = 1; p.s.Kd = p.Kd; p.s.SK = (p.Kd + 63) / 64;
  p.s.x_hi = p.x_hi; p.s.x_lo = p.x_lo; p.s.ldx = p.ldx; p.s.M = p.M;
  if (MP == 8) return (p.Kd % 1024 == 0) ? launch_lm_t<1, 1, 16, true>(p, st) : launch_lm_t<1, 1, 16, false>(p, st);
  if (MP == 32) return (p.Kd % 1024 == 0) ? launch_lm_t<4, 2, 16, true>(p, st) : launch_lm_t<4, 2, 16, false>(p, st);
  return (p.Kd % 512 == 0) ? launch_lm_t<16, 1, 8, true>(p, st) : launch_lm_t<16, 1, 8, false>(p, st);
}

}  // namespace dart
