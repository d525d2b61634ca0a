// Dense projections of the draft-side prefill (Section 3.2: the draft layer's KV cache of the prefix):
//   feature FC       g[T, h]      = f[T, 3h] W_fc^T          -> z_g = bf16(g * gain_g), per-row sums of squares
//   k / v projection y[T, Hkv dh] = rstd_g (z_g W^g^T) + z_e W^e^T, RoPE on k, stored into the KV cache
// for T new prefix rows at once.  Unlike the drafting step (8..128 token rows against the whole model, HBM-bound)
// this is a compute-bound GEMM, so the operands swap sides: 128 token rows are the M side of tcgen05.mma, 256
// output features its N side, K = 16, four per 64-k stage; both operand tiles arrive by TMA (128-byte swizzle) in
// a shared-memory ring (16 KB + 32 KB per stage, four stages; the FC's pair items: 2 x 16 KB + 32 KB, three), the
// fp32 accumulators sit in tensor memory (FC: two buffers of 256 columns -- a single tile's read-out overlaps the
// next tile's MMAs, a pair item fills both; k/v: one buffer per half of z, because the two halves carry different
// 1/rms factors), and four warps read them out, one token row per thread.
// One persistent CTA per SM walks its list of work items (below); every mbarrier wait is bounded.
#include "common.cuh"
#include "kernels.h"
#include "umma.cuh"

namespace dart {

using namespace umma;

constexpr int kDenseThreads = 256;
constexpr int kDenseABytes = 128 * 64 * 2, kDenseBBytes = 256 * 64 * 2;
// The ring holds 192 KB either way: four stages of one token tile + one weight tile (48 KB), or -- feature FC with
// pairs of token tiles -- three of two token tiles + one weight tile (64 KB).
constexpr int kDenseRingBytes = 192 * 1024;
constexpr size_t kDenseSmem = (size_t)kDenseRingBytes + 1024;

// Work items.  A 128 x 256 tile asks for 48 KB of operands per 512 cycles of MMAs, more than an SM is delivered, so
// the feature FC (mode 0) runs whole waves of PAIR items first: two token tiles that share the weight tile of a stage
// (64 KB per 1024 cycles of MMAs), one accumulator each -- which leaves no second buffer to overlap the read-out with
// the next item, a few per cent of an item with K = 3h.  What does not fill a wave of pairs runs as single tiles.
// CTA c takes pair items c, c + G, ... of the first `pair_waves` * G pairs, then single tiles c, c + G, ... of the rest:
// the two halves of every remaining pair (neighbouring CTAs share its weight tile in L2), then an odd last row of
// token tiles.  Every role of a CTA walks the same list.
struct DenseItem { int mt, nm, nt; };
__device__ __forceinline__ bool dense_item(const DenseArgs& a, int i, int m_tiles, int n_tiles, DenseItem& it) {
  const int G = gridDim.x, c = blockIdx.x;
  const int pairs = (m_tiles >> 1) * n_tiles, n_pair = a.pair_waves * G;     // host: n_pair <= pairs
  if (i < a.pair_waves) {
    const int bi = i * G + c;
    it.mt = 2 * (bi / n_tiles); it.nm = 2; it.nt = bi % n_tiles;
    return true;
  }
  const int si = (i - a.pair_waves) * G + c, split = 2 * (pairs - n_pair);
  if (si < split) {
    const int bi = n_pair + (si >> 1);
    it.mt = 2 * (bi / n_tiles) + (si & 1); it.nm = 1; it.nt = bi % n_tiles;
    return true;
  }
  if ((m_tiles & 1) && si - split < n_tiles) {
    it.mt = m_tiles - 1; it.nm = 1; it.nt = si - split;
    return true;
  }
  return false;
}

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
  __shared__ uint64_t full[4], empty[4], acc_full[2], acc_empty[2];
  __shared__ uint32_t tmem_base;
  __shared__ int abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m_tiles = (a.T + 127) >> 7, n_tiles = a.n_w * a.n_tiles_per_w;
  const int KBt = a.KB[0] + a.KB[1];            // k-blocks per tile (k/v: g half then e half)
  const bool two_acc = a.mode == 1;             // k/v: one accumulator per half of z, no double buffering
  const int stages = a.pair_waves > 0 ? 3 : 4;
  const int stage_bytes = kDenseRingBytes / stages, w_off = stage_bytes - kDenseBBytes;   // [A0 | (A1) | W]

  if (threadIdx.x == 0) {
    for (int s = 0; s < 4; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
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
  // The feature FC lets its successor start at once: that is prefill_embed_kernel, a few small blocks per SM that fit
  // beside this CTA, share nothing with it (the other half of z) and wait for this grid before they exit.
  if (a.mode == 0) pdl_trigger();

  // Accumulator buffers of an item, the same in the MMA thread and the read-out warps: k/v items use both halves
  // under buffer 0's barriers; a pair item takes buffers 0 and 1; a single FC tile takes them in turn.
  if (warp == 0 && lane == 0) {
    // ---- producer
    int s = 0, ph = 0;
    bool ok = true;
    DenseItem it;
    for (int i = 0; ok && dense_item(a, i, m_tiles, n_tiles, it); ++i) {
      const int w = it.nt / a.n_tiles_per_w, nrow = (it.nt - w * a.n_tiles_per_w) * 256;
      for (int kb = 0; kb < KBt; ++kb) {
        if (ph > 0 && !mbar_wait(&empty[s], (ph - 1) & 1, &abort_flag)) { ok = false; break; }
        const int half = kb < a.KB[0] ? 0 : 1, kk = (half ? kb - a.KB[0] : kb) * 64;
        uint8_t* st = ring + (size_t)s * stage_bytes;
        mbar_expect_tx(&full[s], it.nm * kDenseABytes + kDenseBBytes);
        tma_load_2d(st, &a.mapA, &full[s], a.a_koff[half] + kk, it.mt * 128);
        if (it.nm == 2) tma_load_2d(st + kDenseABytes, &a.mapA, &full[s], a.a_koff[half] + kk, (it.mt + 1) * 128);
        tma_load_2d(st + w_off, &a.mapW[w * 2 + half], &full[s], kk, nrow);
        if (++s == stages) { s = 0; ++ph; }
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer
    constexpr uint32_t idesc = idesc_bf16(128, 256);
    int s = 0, ph = 0, use[2] = {0, 0}, tog = 0;
    bool ok = true;
    DenseItem it;
    for (int i = 0; ok && dense_item(a, i, m_tiles, n_tiles, it); ++i) {
      const int b0 = (two_acc || it.nm == 2) ? 0 : tog, nb = (!two_acc && it.nm == 2) ? 2 : 1;
      if (!two_acc && it.nm == 1) tog ^= 1;
      for (int b = b0; b < b0 + nb && ok; ++b)
        if (use[b] > 0) {
          if (!mbar_wait(&acc_empty[b], (use[b] - 1) & 1, &abort_flag)) ok = false;
        }
      if (!ok) break;
      tc_fence_after();
      for (int kb = 0; kb < KBt; ++kb) {
        if (!mbar_wait(&full[s], ph & 1, &abort_flag)) { ok = false; break; }
        tc_fence_after();
        const int half = kb < a.KB[0] ? 0 : 1;
        const bool first = kb == 0 || kb == a.KB[0];
        const uint32_t acc = tmem + (two_acc ? half * 256 : b0 * 256);
        const uint32_t wa = smem_u32(ring + (size_t)s * stage_bytes);
        const uint64_t ad = desc_sw128(wa), bd = desc_sw128(wa + w_off);
        if (it.nm == 2) {
          const uint64_t ad1 = desc_sw128(wa + kDenseABytes);
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            mma_f16(acc, ad + 2 * k, bd + 2 * k, idesc, (!first || k > 0) ? 1u : 0u);
            mma_f16(acc + 256, ad1 + 2 * k, bd + 2 * k, idesc, (!first || k > 0) ? 1u : 0u);
          }
        } else {
#pragma unroll
          for (int k = 0; k < 4; ++k) mma_f16(acc, ad + 2 * k, bd + 2 * k, idesc, (!first || k > 0) ? 1u : 0u);
        }
        mma_commit(&empty[s]);
        if (++s == stages) { s = 0; ++ph; }
      }
      if (ok)
        for (int b = b0; b < b0 + nb; ++b) { mma_commit(&acc_full[b]); ++use[b]; }
    }
  } else if (warp >= 4) {
    // ---- read-out: TMEM lane = token row of the tile, columns = output features
    const int wq = warp & 3, row = wq * 32 + lane;
    int use[2] = {0, 0}, tog = 0;
    bool ok = true;
    DenseItem it;
    for (int i = 0; ok && dense_item(a, i, m_tiles, n_tiles, it); ++i) {
      const int b0 = (two_acc || it.nm == 2) ? 0 : tog, nb = (!two_acc && it.nm == 2) ? 2 : 1;
      if (!two_acc && it.nm == 1) tog ^= 1;
     for (int buf = b0; buf < b0 + nb; ++buf) {
      const int mt = it.mt + (buf - b0), nt = it.nt;
      if (!mbar_wait(&acc_full[buf], use[buf] & 1, &abort_flag)) { ok = false; break; }
      ++use[buf];
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
  }
  pdl_trigger();
  __syncthreads();
  if (warp == 2) { tc_fence_after(); tmem_dealloc(tmem, 512); }
  if (abort_flag && threadIdx.x == 0) {
    atomicExch(a.status, DEV_TIMEOUT);
    for (int i = 0; i < 100; ++i) __nanosleep(1000);
  }
}

// z e-half of the prefill rows: RMSNorm of the next token's embedding, gain-scaled, bf16.  A row is read and written
// 16 bytes per thread and request when h is a multiple of 8 (two-byte requests made this kernel 64 us for 4096 rows
// of 5120: a tenth of the prefill).  Launched right AFTER the feature FC, which triggers its dependents at once: a
// few blocks per SM walk the rows while the FC's CTAs compute (its inputs are the caller's; the half of z it writes
// is read by the k / v kernel only, and the previous pass's k / v kernel was complete before the FC triggered).  It
// waits for the FC's grid at its END, so that the k / v kernel, which waits for this grid, finds both halves of z.
__global__ void __launch_bounds__(256) prefill_embed_kernel(const int32_t* tokens, int T, int vocab, const bf16* embed, const bf16* gain_e,
                                                            int h, float eps, bf16* z, long long ldz) {
  __shared__ float sh[32];
 for (int t = blockIdx.x; t < T; t += gridDim.x) {
  const int id = min(max(tokens[t], 0), vocab - 1);
  const bf16* row = embed + (size_t)id * h;
  bf16* out = z + (size_t)t * ldz + h;
  const bool vec = (h & 7) == 0 && ((reinterpret_cast<uintptr_t>(row) | reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(gain_e)) & 15) == 0;
  float ss = 0.f;
  if (vec) {
    for (int n = threadIdx.x; n < (h >> 3); n += blockDim.x) {
      const uint4 q = __ldg(reinterpret_cast<const uint4*>(row) + n);
      const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&q);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 f = __bfloat1622float2(p2[j]);
        ss += f.x * f.x + f.y * f.y;
      }
    }
  } else {
    for (int n = threadIdx.x; n < h; n += blockDim.x) {
      const float v = __bfloat162float(row[n]);
      ss += v * v;
    }
  }
  ss = block_sum(ss, sh);
  const float rs = 1.f / sqrtf(ss / (float)h + eps);
  if (vec) {
    for (int n = threadIdx.x; n < (h >> 3); n += blockDim.x) {
      const uint4 q = __ldg(reinterpret_cast<const uint4*>(row) + n), g = __ldg(reinterpret_cast<const uint4*>(gain_e) + n);
      const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&q);
      const __nv_bfloat162* g2 = reinterpret_cast<const __nv_bfloat162*>(&g);
      uint32_t w[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 f = __bfloat1622float2(p2[j]), gg = __bfloat1622float2(g2[j]);
        // the same products, in the same order, as the element-wise form: (x * rs) * gain, rounded once
        const __nv_bfloat162 v = __floats2bfloat162_rn(f.x * rs * gg.x, f.y * rs * gg.y);
        w[j] = *reinterpret_cast<const uint32_t*>(&v);
      }
      reinterpret_cast<uint4*>(out)[n] = make_uint4(w[0], w[1], w[2], w[3]);
    }
  } else {
    for (int n = threadIdx.x; n < h; n += blockDim.x)
      out[n] = __float2bfloat16(__bfloat162float(row[n]) * rs * __bfloat162float(gain_e[n]));
  }
  __syncthreads();    // sh is reused by the next row's sum
 }
  pdl_wait();
  pdl_trigger();
}

cudaError_t launch_prefill_embed(const int32_t* tokens, int T, int vocab, const bf16* embed, const bf16* gain_e, int h, float eps,
                                 bf16* z, long long ldz, int n_sm, cudaStream_t st) {
  const int blocks = T < 2 * n_sm ? T : 2 * n_sm;   // what fits beside a CTA of the feature FC (registers)
  return launch_pdl(prefill_embed_kernel, dim3(blocks), dim3(256), 0, st, tokens, T, vocab, embed, gain_e, h, eps, z, ldz);
}

cudaError_t launch_umma_dense(const DenseArgs& a, int n_sm, cudaStream_t st) {
  const cudaError_t e = allow_dynamic_smem(reinterpret_cast<const void*>(umma_dense_kernel), kDenseSmem);
  if (e != cudaSuccess) return e;
  const int m_tiles = (a.T + 127) / 128, n_tiles = a.n_w * a.n_tiles_per_w, tiles = m_tiles * n_tiles;
  const int grid = tiles < n_sm ? tiles : n_sm;
  DenseArgs b = a;
  b.pair_waves = 0;
  if (a.mode == 0) {
    // whole waves of pair items, as many as make the estimate smallest: a pair item costs two single tiles' MMAs,
    // a single tile a quarter more than its own (the operands arrive more slowly than the MMAs take them)
    const int pairs = (m_tiles / 2) * n_tiles;
    double best = 0.0;
    for (int pw = 0; pw <= pairs / grid; ++pw) {
      const int singles = tiles - 2 * pw * grid;
      const double t = 2.0 * pw + 1.25 * ((singles + grid - 1) / grid);
      if (pw == 0 || t < best) { best = t; b.pair_waves = pw; }
    }
  }
  return launch_pdl(umma_dense_kernel, dim3(grid), dim3(kDenseThreads), kDenseSmem, st, b);
}

}  // namespace dart
