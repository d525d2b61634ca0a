// LM head with fused vocab-sharded log-softmax + per-position top-k
// (Section 3.2: one logit row per future position; Algorithm 1 lines 6-8; Appendix D s_logit).
//
// The LM head is 63 % of the step's bytes at the Qwen3-14B shape, so it is the kernel the
// roofline is quoted on.  Each CTA owns a contiguous range of 16-row vocab tiles, balanced to
// within one tile.  Inside a tile the eight warps split the reduction dimension (warp w takes
// k-steps w, w+8, ...), stream their weight fragments global -> registers with 128-bit loads
// (same operand mapping as the projections' kernel), and the eight partial tiles are summed
// through shared memory.  Complete logits never leave the SM: every 128 vocab rows a warp per
// token row folds them into a running (max, sum-exp) pair and an exact top-32 list held one
// entry per lane.  The CTA writes (max, sum-exp, list) per token row; topk_merge_kernel
// (topk_merge.cu) combines the CTAs' results and emits the k best ids with s_logit = log(softmax + eps).
//
// With temperature > 0 the list is ordered by logit/T + Gumbel noise (Gumbel-top-k = sampling
// without replacement); the noise of token v in row (b, r) is word v&3 of
// Philox4x32-10(counter = (v>>2, r, b, step), key = seed).
#include "common.cuh"
#include "kernels.h"

namespace dart {

struct LmCursor {
  int mt, i;  // vocab tile, index of this warp's k-step inside the tile
};

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

// FULL: Kd is a multiple of 512 (every warp has the same number of whole k-steps) and all MP
// token rows are valid, so the streaming loop carries no bounds predicates at all.
template <int NT, bool HAS_LO, int PF, bool FULL>
__global__ void __launch_bounds__(256, (NT <= 4 ? 2 : 1)) lm_head_kernel(const LmParams p) {
  constexpr int MP = 8 * NT;
  constexpr int RB = (NT <= 4) ? 2 : 1;      // reduce buffers
  constexpr int SROW = 128 + 1;              // stage row stride (floats)
  extern __shared__ __align__(16) float sm[];
  float* red = sm;                           // [RB][8 warps][16][MP]
  float* stage = red + RB * 8 * 16 * MP;     // [MP][SROW]
  float* st_key = stage + MP * SROW;         // [MP][32]
  float* st_y = st_key + MP * 32;
  int* st_id = reinterpret_cast<int*>(st_y + MP * 32);
  float* st_ms = reinterpret_cast<float*>(st_id + MP * 32);  // [MP][2]
  float* s_rstd = st_ms + 2 * MP;                            // [MP] 1/rms of the final RMSNorm per token row

  const int c = blockIdx.x, G = gridDim.x;
  const int n_mt = p.V >> 4;
  const int mt0 = (int)(((long long)c * n_mt) / G), mt1 = (int)(((long long)(c + 1) * n_mt) / G);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int SK = (p.Kd + 63) >> 6;
  const int spw = (SK + 7) >> 3;  // k-steps per warp per tile

  for (int i = tid; i < MP * 32; i += 256) { st_key[i] = -INFINITY; st_y[i] = 0.f; st_id[i] = 0x7fffffff; }
  for (int i = tid; i < MP; i += 256) {
    st_ms[2 * i] = -INFINITY;
    st_ms[2 * i + 1] = 0.f;
    float ssq = 0.f;  // the activations are x * gain; their 1/rms multiplies the logits (same fixed order everywhere)
    if (i < p.M)
      for (int tl = 0; tl < p.ss_tiles; ++tl) ssq += p.ss_in[(size_t)tl * p.ss_mp + i];
    s_rstd[i] = i < p.M ? 1.f / sqrtf(ssq / (float)p.Kd + p.rms_eps) : 0.f;
  }
  __syncthreads();

  float acc[NT][4];
#pragma unroll
  for (int n = 0; n < NT; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
  uint4 a[PF][4];
  LmCursor ld{mt0, 0}, cp{mt0, 0};
  const int nsteps = (mt1 - mt0) * spw;

  auto issue = [&](uint4(&dst)[4]) {
    const int ks = warp + 8 * ld.i;
    const int ka = ks * 64 + chunk_k0(t), kb = ks * 64 + chunk_k1(t);
    const bf16* r0 = p.W + (size_t)(ld.mt * 16 + g) * p.Kd;
    const bf16* r1 = r0 + (size_t)8 * p.Kd;
    if (FULL) {
      dst[0] = ld_stream16(r0 + ka);
      dst[1] = ld_stream16(r0 + kb);
      dst[2] = ld_stream16(r1 + ka);
      dst[3] = ld_stream16(r1 + kb);
    } else {
      const bool va = ks < SK && ka < p.Kd, vb = ks < SK && kb < p.Kd;
      const uint4 z = make_uint4(0, 0, 0, 0);
      dst[0] = va ? ld_stream16(r0 + ka) : z;
      dst[1] = vb ? ld_stream16(r0 + kb) : z;
      dst[2] = va ? ld_stream16(r1 + ka) : z;
      dst[3] = vb ? ld_stream16(r1 + kb) : z;
    }
    if (++ld.i == spw) { ld.i = 0; ++ld.mt; }
  };

#pragma unroll
  for (int s = 0; s < PF; ++s)
    if (s < nsteps) issue(a[s]);

  int buf = 0;
  for (int u = 0; u < nsteps; u += PF) {
#pragma unroll
    for (int s = 0; s < PF; ++s) {
      if (u + s < nsteps) {
        const int ks = warp + 8 * cp.i;
        const int ka = ks * 64 + chunk_k0(t), kb = ks * 64 + chunk_k1(t);
        const bool kval = (ks < SK) && (ka < p.Kd), kval2 = (ks < SK) && (kb < p.Kd);
        const uint32_t w0[8] = {a[s][0].x, a[s][0].y, a[s][0].z, a[s][0].w, a[s][1].x, a[s][1].y, a[s][1].z, a[s][1].w};
        const uint32_t w1[8] = {a[s][2].x, a[s][2].y, a[s][2].z, a[s][2].w, a[s][3].x, a[s][3].y, a[s][3].z, a[s][3].w};
#pragma unroll
        for (int n = 0; n < NT; ++n) {
          const int tok = n * 8 + g;
          uint4 h0 = make_uint4(0, 0, 0, 0), h1 = h0, l0 = h0, l1 = h0;
          const bf16* xp = p.x_hi + (size_t)tok * p.ldx;
          const bf16* xq = p.x_lo + (size_t)tok * p.ldx;
          if (FULL) {
            h0 = ld_act16(xp + ka);
            h1 = ld_act16(xp + kb);
            if (HAS_LO) { l0 = ld_act16(xq + ka); l1 = ld_act16(xq + kb); }
          } else if (tok < p.M) {
            if (kval) {
              h0 = ld_act16(xp + ka);
              if (HAS_LO) l0 = ld_act16(xq + ka);
            }
            if (kval2) {
              h1 = ld_act16(xp + kb);
              if (HAS_LO) l1 = ld_act16(xq + kb);
            }
          }
          const uint32_t xh[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
          const uint32_t xl[8] = {l0.x, l0.y, l0.z, l0.w, l1.x, l1.y, l1.z, l1.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            mma_bf16_16816(acc[n], w0[2 * j], w1[2 * j], w0[2 * j + 1], w1[2 * j + 1], xh[2 * j], xh[2 * j + 1]);
            if (HAS_LO)
              mma_bf16_16816(acc[n], w0[2 * j], w1[2 * j], w0[2 * j + 1], w1[2 * j + 1], xl[2 * j], xl[2 * j + 1]);
          }
        }
        if (u + s + PF < nsteps) issue(a[s]);

        if (cp.i == spw - 1) {
          // ---- end of a vocab tile: cross-warp reduction of the eight k-slices
          float* rw = red + ((size_t)buf * 8 + warp) * 16 * MP;
#pragma unroll
          for (int n = 0; n < NT; ++n) {
            *reinterpret_cast<float2*>(rw + g * MP + n * 8 + 2 * t) = make_float2(acc[n][0], acc[n][1]);
            *reinterpret_cast<float2*>(rw + (g + 8) * MP + n * 8 + 2 * t) = make_float2(acc[n][2], acc[n][3]);
            acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
          }
          __syncthreads();
          const int slot = (cp.mt - mt0) & 7;
          for (int e = tid; e < 16 * MP; e += 256) {
            const int row = e / MP, tok = e % MP;
            float v = 0.f;
#pragma unroll
            for (int w = 0; w < 8; ++w) v += red[((size_t)buf * 8 + w) * 16 * MP + row * MP + tok];
            v *= s_rstd[tok];
            stage[tok * SROW + slot * 16 + row] = v;
            if (p.logits_out != nullptr && tok < p.M) p.logits_out[(size_t)tok * p.V + cp.mt * 16 + row] = v;
          }
          if (RB == 1) __syncthreads();
          buf = (RB == 2) ? (buf ^ 1) : 0;

          if (slot == 7 || cp.mt == mt1 - 1) {
            // ---- fold up to 128 complete logits per token row into the running softmax / top-k state
            __syncthreads();
            const int nrows = (slot + 1) * 16;
            const int id0 = (cp.mt - slot) * 16;
            for (int tk = warp; tk < p.M; tk += 8) {
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
        if (++cp.i == spw) { cp.i = 0; ++cp.mt; }
      }
    }
  }
  __syncthreads();
  for (int i = tid; i < MP * 32; i += 256) {
    const size_t o = (size_t)c * MP * 32 + i;
    p.part_key[o] = st_key[i];
    p.part_y[o] = st_y[i];
    p.part_id[o] = st_id[i];
  }
  for (int i = tid; i < MP * 2; i += 256) p.part_stats[(size_t)c * MP * 2 + i] = st_ms[i];
}

template <int NT>
static size_t lm_smem_bytes() {
  constexpr int MP = 8 * NT, RB = (NT <= 4) ? 2 : 1;
  return sizeof(float) * ((size_t)RB * 8 * 16 * MP + (size_t)MP * 129 + 3 * (size_t)MP * 32 + 3 * (size_t)MP);
}

template <int NT, int PF, bool FULL>
static cudaError_t launch_lm_t(const LmParams& p, cudaStream_t st) {
  const size_t smem = lm_smem_bytes<NT>();
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(lm_head_kernel<NT, true, PF, FULL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  lm_head_kernel<NT, true, PF, FULL><<<p.grid, 256, smem, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_lm_head(const LmParams& p, cudaStream_t st) {
  const int MP = padded_tokens(p.M);
  if (p.x_lo == nullptr) return cudaErrorInvalidValue;  // the LM head always takes hi + lo activations
  const bool full = (p.Kd % 512 == 0) && (p.M == MP);
  if (MP == 8) return full ? launch_lm_t<1, 4, true>(p, st) : launch_lm_t<1, 4, false>(p, st);
  if (MP == 32) return full ? launch_lm_t<4, 2, true>(p, st) : launch_lm_t<4, 2, false>(p, st);
  return full ? launch_lm_t<16, 2, true>(p, st) : launch_lm_t<16, 2, false>(p, st);
}

}  // namespace dart
