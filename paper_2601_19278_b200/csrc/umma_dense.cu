// Dense projections of the draft-side prefill (Section 3.2: the draft layer's KV cache of the prefix):
//   feature FC       g[T, h]      = f[T, 3h] W_fc^T          -> z_g = bf16(g * gain_g), per-row sums of squares
//   k / v projection y[T, Hkv dh] = rstd_g (z_g W^g^T) + z_e W^e^T, RoPE on k, stored into the KV cache
// for T new prefix rows at once.  Unlike the drafting step (8..128 token rows against the whole model, HBM-bound)
// this is a compute-bound GEMM, so the operands swap sides: 128 token rows are the M side of tcgen05.mma, 256
// output features its N side, K = 16, four per 64-k stage; both operand tiles arrive by TMA (128-byte swizzle) in
// a four-stage shared-memory ring (16 KB + 32 KB per stage), the fp32 accumulators sit in tensor memory (FC: two
// buffers of 256 columns, so a tile's read-out overlaps the next tile's MMAs; k/v: one buffer per half of z,
// because the two halves carry different 1/rms factors), and four warps read them out, one token row per thread.
// One persistent CTA per SM walks the (token tile, feature tile) space; every mbarrier wait is bounded.
#include "common.cuh"
#include "kernels.h"
#include "umma.cuh"

namespace dart {

using namespace umma;

constexpr int kDenseThreads = 256;
constexpr int kDenseStages = 4;
constexpr int kDenseABytes = 128 * 64 * 2, kDenseBBytes = 256 * 64 * 2, kDenseStageBytes = kDenseABytes + kDenseBBytes;
constexpr size_t kDenseSmem = (size_t)kDenseStages * kDenseStageBytes + 1024;

// Cache slab and absolute position of packed row t (rows of sequence b are seq_off[b] .. seq_off[b+1]-1).
__device__ __forceinline__ void row_place(const DenseArgs& a, int t, int& slab, int& pos) {
  int b = 0;
  while (b + 1 < a.B && t >= a.seq_off[b + 1]) ++b;
  slab = b;
  pos = a.seq_P[b] + (t - a.seq_off[b]);
}

__global__ void __launch_bounds__(kDenseThreads, 1) umma_dense_kernel(const __grid_constant__ DenseArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ uint64_t full[kDenseStages], empty[kDenseStages], acc_full[2], acc_empty[2];
  __shared__ uint32_t tmem_base;
  __shared__ int abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m_tiles = (a.T + 127) >> 7, n_tiles = a.n_w * a.n_tiles_per_w, tiles = m_tiles * n_tiles;
  const int KBt = a.KB[0] + a.KB[1];            // k-blocks per tile (k/v: g half then e half)
  const bool two_acc = a.mode == 1;             // k/v: one accumulator per half of z, no double buffering

  if (threadIdx.x == 0) {
    for (int s = 0; s < kDenseStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 128); }
    abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 2) tmem_alloc(&tmem_base, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base;
  pdl_wait();   // every operand of this kernel is produced by the kernels before it

  if (warp == 0 && lane == 0) {
    // ---- producer
    int s = 0, ph = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < tiles && ok; t += gridDim.x) {
      const int mt = t / n_tiles, nt = t - mt * n_tiles;
      const int w = nt / a.n_tiles_per_w, nrow = (nt - w * a.n_tiles_per_w) * 256;
      for (int kb = 0; kb < KBt; ++kb) {
        if (ph > 0 && !mbar_wait(&empty[s], (ph - 1) & 1, &abort_flag)) { ok = false; break; }
        const int half = kb < a.KB[0] ? 0 : 1, kk = (half ? kb - a.KB[0] : kb) * 64;
        uint8_t* st = ring + (size_t)s * kDenseStageBytes;
        mbar_expect_tx(&full[s], kDenseStageBytes);
        tma_load_2d(st, &a.mapA, &full[s], a.a_koff[half] + kk, mt * 128);
        tma_load_2d(st + kDenseABytes, &a.mapW[w * 2 + half], &full[s], kk, nrow);
        if (++s == kDenseStages) { s = 0; ++ph; }
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer
    constexpr uint32_t idesc = idesc_bf16(128, 256);
    int s = 0, ph = 0, it = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < tiles && ok; t += gridDim.x, ++it) {
      const int buf = two_acc ? 0 : (it & 1), use = two_acc ? it : (it >> 1);
      if (use > 0) {
        if (!mbar_wait(&acc_empty[buf], (use - 1) & 1, &abort_flag)) break;
        tc_fence_after();
      }
      for (int kb = 0; kb < KBt; ++kb) {
        if (!mbar_wait(&full[s], ph & 1, &abort_flag)) { ok = false; break; }
        tc_fence_after();
        const int half = kb < a.KB[0] ? 0 : 1;
        const bool first = kb == 0 || kb == a.KB[0];
        const uint32_t acc = tmem + (two_acc ? half * 256 : buf * 256);
        const uint32_t wa = smem_u32(ring + (size_t)s * kDenseStageBytes);
        const uint64_t ad = desc_sw128(wa), bd = desc_sw128(wa + kDenseABytes);
#pragma unroll
        for (int k = 0; k < 4; ++k) mma_f16(acc, ad + 2 * k, bd + 2 * k, idesc, (!first || k > 0) ? 1u : 0u);
        mma_commit(&empty[s]);
        if (++s == kDenseStages) { s = 0; ++ph; }
      }
      if (ok) mma_commit(&acc_full[buf]);
    }
  } else if (warp >= 4) {
    // ---- read-out: TMEM lane = token row of the tile, columns = output features
    const int wq = warp & 3, row = wq * 32 + lane;
    int it = 0;
    for (int t = blockIdx.x; t < tiles; t += gridDim.x, ++it) {
      const int mt = t / n_tiles, nt = t - mt * n_tiles;
      const int buf = two_acc ? 0 : (it & 1), use = two_acc ? it : (it >> 1);
      if (!mbar_wait(&acc_full[buf], use & 1, &abort_flag)) break;
      tc_fence_after();
      const int tok = mt * 128 + row;
      const bool live = tok < a.T;
      const uint32_t tb = tmem + ((uint32_t)(wq * 32) << 16);
      if (a.mode == 0) {
        // feature FC: z_g = bf16(g * gain), and this tile's share of the row's sum of squares
        const int n0 = nt * 256;
        float ssq = 0.f;
#pragma unroll 1
        for (int c = 0; c < 256; c += 16) {
          uint32_t r[16];
          tmem_ld16(tb + buf * 256 + c, r);
          tmem_ld_wait();
          if (live && n0 + c < a.n_out) {
            uint32_t packed[8];
#pragma unroll
            for (int j = 0; j < 16; j += 2) {
              const float g0 = __uint_as_float(r[j]), g1 = __uint_as_float(r[j + 1]);
              ssq += g0 * g0 + g1 * g1;
              const __nv_bfloat162 v = __floats2bfloat162_rn(g0 * __bfloat162float(a.gain[n0 + c + j]), g1 * __bfloat162float(a.gain[n0 + c + j + 1]));
              packed[j >> 1] = *reinterpret_cast<const uint32_t*>(&v);
            }
            uint4* dst = reinterpret_cast<uint4*>(a.z + (size_t)tok * a.ldz + n0 + c);
            dst[0] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
            dst[1] = make_uint4(packed[4], packed[5], packed[6], packed[7]);
          }
        }
        if (live) a.ss[(size_t)tok * a.ss_ld + nt] = ssq;
      } else {
        // k / v: y = rstd_g * (g half) + (e half); RoPE on k; bf16 into the cache row of this token
        float rstd = 0.f;
        int slab = 0, pos = 0;
        if (live) {
          float s2 = 0.f;
          for (int j = 0; j < a.ss_n; ++j) s2 += a.ss[(size_t)tok * a.ss_ld + j];
          rstd = 1.f / sqrtf(s2 / (float)a.h + a.eps);
          row_place(a, tok, slab, pos);
        }
        const int w = nt / a.n_tiles_per_w, feat0 = (nt - w * a.n_tiles_per_w) * 256;   // w: 0 = k, 1 = v
        const int dh = a.dh, half = dh >> 1;
        bf16* cache = w == 0 ? a.k_cache : a.v_cache;
#pragma unroll 1
        for (int hd = 0; hd < 256 / dh; ++hd) {
          const int head = feat0 / dh + hd;
#pragma unroll 1
          for (int c = 0; c < half; c += 16) {
            uint32_t g1[16], g2[16], e1[16], e2[16];
            tmem_ld16(tb + hd * dh + c, g1);
            tmem_ld16(tb + hd * dh + half + c, g2);
            tmem_ld16(tb + 256 + hd * dh + c, e1);
            tmem_ld16(tb + 256 + hd * dh + half + c, e2);
            tmem_ld_wait();
            if (live && head < a.Hkv) {
              uint32_t p1[8], p2[8];
#pragma unroll
              for (int j = 0; j < 16; j += 2) {
                float x1[2], x2[2];
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                  const float y1 = rstd * __uint_as_float(g1[j + q]) + __uint_as_float(e1[j + q]);
                  const float y2 = rstd * __uint_as_float(g2[j + q]) + __uint_as_float(e2[j + q]);
                  x1[q] = y1; x2[q] = y2;
                  if (w == 0) {
                    const float2 cs = a.rope_tab[(size_t)pos * half + c + j + q];
                    x1[q] = y1 * cs.x - y2 * cs.y;
                    x2[q] = y2 * cs.x + y1 * cs.y;
                  }
                }
                const __nv_bfloat162 v1 = __floats2bfloat162_rn(x1[0], x1[1]), v2 = __floats2bfloat162_rn(x2[0], x2[1]);
                p1[j >> 1] = *reinterpret_cast<const uint32_t*>(&v1);
                p2[j >> 1] = *reinterpret_cast<const uint32_t*>(&v2);
              }
              bf16* dst = cache + (((size_t)slab * a.Hkv + head) * a.P_cap + pos) * dh;
              reinterpret_cast<uint4*>(dst + c)[0] = make_uint4(p1[0], p1[1], p1[2], p1[3]);
              reinterpret_cast<uint4*>(dst + c)[1] = make_uint4(p1[4], p1[5], p1[6], p1[7]);
              reinterpret_cast<uint4*>(dst + half + c)[0] = make_uint4(p2[0], p2[1], p2[2], p2[3]);
              reinterpret_cast<uint4*>(dst + half + c)[1] = make_uint4(p2[4], p2[5], p2[6], p2[7]);
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(&acc_empty[buf]);
    }
  }
  pdl_trigger();
  __syncthreads();
  if (warp == 2) { tc_fence_after(); tmem_dealloc(tmem, 512); }
  if (abort_flag && threadIdx.x == 0) {
    atomicExch(a.status, DEV_TIMEOUT);
    for (int i = 0; i < 100; ++i) __nanosleep(1000);
  }
}

// z e-half of the prefill rows: RMSNorm of the next token's embedding, gain-scaled, bf16.  One block per row.
__global__ void __launch_bounds__(256) prefill_embed_kernel(const int32_t* tokens, int T, int vocab, const bf16* embed, const bf16* gain_e,
                                                            int h, float eps, bf16* z, long long ldz) {
  __shared__ float sh[32];
  pdl_wait();
  const int t = blockIdx.x;
  const int id = min(max(tokens[t], 0), vocab - 1);
  const bf16* row = embed + (size_t)id * h;
  float ss = 0.f;
  for (int n = threadIdx.x; n < h; n += blockDim.x) {
    const float v = __bfloat162float(row[n]);
    ss += v * v;
  }
  ss = block_sum(ss, sh);
  const float rs = 1.f / sqrtf(ss / (float)h + eps);
  for (int n = threadIdx.x; n < h; n += blockDim.x)
    z[(size_t)t * ldz + h + n] = __float2bfloat16(__bfloat162float(row[n]) * rs * __bfloat162float(gain_e[n]));
  pdl_trigger();
}

cudaError_t launch_prefill_embed(const int32_t* tokens, int T, int vocab, const bf16* embed, const bf16* gain_e, int h, float eps,
                                 bf16* z, long long ldz, cudaStream_t st) {
  return launch_pdl(prefill_embed_kernel, dim3(T), dim3(256), 0, st, tokens, T, vocab, embed, gain_e, h, eps, z, ldz);
}

cudaError_t launch_umma_dense(const DenseArgs& a, int n_sm, cudaStream_t st) {
  const cudaError_t e = allow_dynamic_smem(reinterpret_cast<const void*>(umma_dense_kernel), kDenseSmem);
  if (e != cudaSuccess) return e;
  const int tiles = ((a.T + 127) / 128) * a.n_w * a.n_tiles_per_w;
  const int grid = tiles < n_sm ? tiles : n_sm;
  return launch_pdl(umma_dense_kernel, dim3(grid), dim3(kDenseThreads), kDenseSmem, st, a);
}

}  // namespace dart
