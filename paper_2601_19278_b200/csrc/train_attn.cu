// Forward attention under the prefix-shared training mask (Section 3.3, Appendix B): a packed row of
// `prompt_len` clean positions followed by one block of `draft_len` masked positions per prefix position; block n
// reads prompt slots 0..n and, causally, itself; clean positions read causally.  The mask is block-sparse with a
// regular structure, so no mask tensor exists: a CTA owns 128 query rows of one head --
//   * a clean tile: 128 consecutive prompt slots, or
//   * a masked tile: the blocks of T = 128 / draft_len consecutive prefix positions (T * draft_len rows) --
// and walks exactly the key tiles its rows can see: the clean key tiles up to its last prefix position (only the
// last of them needs a per-row bound) and, for a masked tile, its own 128 slots (same block and causal).
// Flash-attention dataflow on the 5th-generation tensor cores:
//   S = Q K^T       tcgen05.mma, operands by TMA (128-byte swizzle), S in tensor memory, two S buffers
//   P = exp2(S - m) four warps, one query row per thread; bf16 P written to shared memory in the operand layout
//   O += P V        tcgen05.mma with V^T tiles (a small kernel transposes V once), O accumulates in tensor memory
// The running reference maximum m only moves when a tile's maximum exceeds it by more than 2^8, so the O rows are
// rescaled in tensor memory a few times per row instead of once per tile.  Every mbarrier wait is bounded.
#include "common.cuh"
#include "kernels.h"
#include "umma.cuh"

namespace dart {

using namespace umma;

constexpr int kTaThreads = 256;
constexpr int kTaTile = 128 * 128 * 2;                 // one 128 x 128 bf16 operand tile: two 64-column halves
constexpr size_t kTaSmem = (size_t)6 * kTaTile + 1024;  // Q, P, 2 x K, 2 x V^T

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
      "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// V [B*Hkv][L][dh] -> V^T of the clean slots [B*Hkv][dh][ldc] and of the masked slots [B*Hkv][dh][ldm], zero beyond.
__global__ void __launch_bounds__(256) train_attn_transpose_kernel(const bf16* __restrict__ v, bf16* __restrict__ vt_c, bf16* __restrict__ vt_m,
                                                                   int L, int Lp, int dh, int ldc, int ldm) {
  __shared__ bf16 tile[32][34];
  const int head = blockIdx.z, region = blockIdx.y & 1, d0 = (blockIdx.y >> 1) * 32, s0 = blockIdx.x * 32;
  const int ld = region ? ldm : ldc, n_src = region ? L - Lp : Lp, src0 = region ? Lp : 0;
  if (s0 >= ld) return;
  bf16* dst = (region ? vt_m : vt_c) + (size_t)head * dh * ld;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int r = ty; r < 32; r += 8) {
    const int s = s0 + r;
    tile[r][tx] = s < n_src ? v[((size_t)head * L + src0 + s) * dh + d0 + tx] : __float2bfloat16(0.f);
  }
  __syncthreads();
  for (int r = ty; r < 32; r += 8)
    if (s0 + tx < ld) dst[(size_t)(d0 + r) * ld + s0 + tx] = tile[tx][r];
}

__global__ void __launch_bounds__(kTaThreads, 1) train_attn_kernel(const __grid_constant__ TrainAttnArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = sm;
  uint8_t* sP = sm + kTaTile;
  uint8_t* sK = sm + 2 * kTaTile;     // two stages
  uint8_t* sV = sm + 4 * kTaTile;     // two stages
  __shared__ uint64_t q_full, k_full[2], k_empty[2], v_full[2], v_empty[2], s_full[2], s_empty[2], p_full, pv_done;
  __shared__ uint32_t tmem_base;
  __shared__ int abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.z, hq = blockIdx.y, hk = hq / (a.Hq / a.Hkv);
  const int Lp = a.prompt_len, d = a.draft_len, L = Lp * (1 + d), T = train_attn_positions_per_tile(d);
  const int n_mask_tiles = (Lp + T - 1) / T, S = a.seq_len[b];
  // heavy tiles first: masked tiles from the last prefix position down, then clean tiles from the last down
  const bool masked = (int)blockIdx.x < n_mask_tiles;
  const int ti = masked ? n_mask_tiles - 1 - (int)blockIdx.x : a.n_clean_tiles - 1 - ((int)blockIdx.x - n_mask_tiles);
  const int n0 = masked ? ti * T : ti * 128;                       // first prefix position / prompt slot of the tile
  const int q_slot0 = masked ? Lp + n0 * d : n0;                   // first packed slot of the tile's query rows
  // a TMA load starts on a 16-byte boundary: the tile's own keys are fetched from the 8-slot boundary below its
  // first masked slot, `shift` columns early
  const int own0 = (n0 * d) & ~7, shift = n0 * d - own0;
  const int rows = masked ? min(T, Lp - n0) * d : min(128, Lp - n0);
  const int last_pos = masked ? min(n0 + T, Lp) - 1 : min(n0 + 128, Lp) - 1;
  const int n_clean = n0 < S ? min(last_pos, S - 1) / 128 + 1 : 0;   // clean key tiles some valid row can see
  const int n_kt = n0 < S ? n_clean + (masked ? 1 : 0) : 0;          // + the tile's own slots
  bf16* out = a.out + ((size_t)(b * a.Hq + hq) * L + q_slot0) * 128;

  if (n_kt == 0) {   // every row lies past the sequence's length: zero rows, nothing to read
    for (int e = threadIdx.x; e < rows * 16; e += kTaThreads) reinterpret_cast<uint4*>(out)[e] = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  if (threadIdx.x == 0) {
    mbar_init(&q_full, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1); mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1);
      mbar_init(&s_full[s], 1); mbar_init(&s_empty[s], 128);
    }
    mbar_init(&p_full, 128);
    mbar_init(&pv_done, 1);
    abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 2) tmem_alloc(&tmem_base, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base;          // columns 0..255: two S buffers; 256..383: O

  if (warp == 0 && lane == 0) {
    // ---- producer: Q once, then per key tile K [128 keys][128] and V^T [128][128 keys]
    const int q_row = (b * a.Hq + hq) * L + q_slot0;
    mbar_expect_tx(&q_full, kTaTile);
    tma_load_2d(sQ, &a.mapQ, &q_full, 0, q_row);
    tma_load_2d(sQ + kTaTile / 2, &a.mapQ, &q_full, 64, q_row);
    for (int j = 0; j < n_kt; ++j) {
      const int s = j & 1;
      const bool own = masked && j == n_kt - 1;
      const int k_row = (b * a.Hkv + hk) * L + (own ? Lp + own0 : j * 128);
      const int v_col = own ? own0 : j * 128, v_row = (b * a.Hkv + hk) * 128;
      if (j >= 2 && !mbar_wait(&k_empty[s], ((j >> 1) - 1) & 1, &abort_flag)) break;
      mbar_expect_tx(&k_full[s], kTaTile);
      tma_load_2d(sK + s * kTaTile, &a.mapK, &k_full[s], 0, k_row);
      tma_load_2d(sK + s * kTaTile + kTaTile / 2, &a.mapK, &k_full[s], 64, k_row);
      if (j >= 2 && !mbar_wait(&v_empty[s], ((j >> 1) - 1) & 1, &abort_flag)) break;
      mbar_expect_tx(&v_full[s], kTaTile);
      const CUtensorMap* mv = own ? &a.mapVm : &a.mapVc;
      tma_load_2d(sV + s * kTaTile, mv, &v_full[s], v_col, v_row);
      tma_load_2d(sV + s * kTaTile + kTaTile / 2, mv, &v_full[s], v_col + 64, v_row);
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer
    constexpr uint32_t idesc = idesc_bf16(128, 128);
    const uint64_t dq0 = desc_sw128(smem_u32(sQ)), dq1 = desc_sw128(smem_u32(sQ + kTaTile / 2));
    const uint64_t dp0 = desc_sw128(smem_u32(sP)), dp1 = desc_sw128(smem_u32(sP + kTaTile / 2));
    bool ok = mbar_wait(&q_full, 0, &abort_flag);
    auto issue_s = [&](int j) -> bool {      // S[j & 1] = Q K_j^T
      const int s = j & 1;
      if (j >= 2 && !mbar_wait(&s_empty[s], ((j >> 1) - 1) & 1, &abort_flag)) return false;
      if (!mbar_wait(&k_full[s], (j >> 1) & 1, &abort_flag)) return false;
      tc_fence_after();
      const uint64_t dk0 = desc_sw128(smem_u32(sK + s * kTaTile)), dk1 = desc_sw128(smem_u32(sK + s * kTaTile + kTaTile / 2));
#pragma unroll
      for (int k = 0; k < 4; ++k) mma_f16(tmem + s * 128, dq0 + 2 * k, dk0 + 2 * k, idesc, k > 0 ? 1u : 0u);
#pragma unroll
      for (int k = 0; k < 4; ++k) mma_f16(tmem + s * 128, dq1 + 2 * k, dk1 + 2 * k, idesc, 1u);
      mma_commit(&k_empty[s]);
      mma_commit(&s_full[s]);
      return true;
    };
    if (ok) ok = issue_s(0);
    for (int j = 0; j < n_kt && ok; ++j) {
      const int s = j & 1;
      if (j + 1 < n_kt && !issue_s(j + 1)) break;
      if (!mbar_wait(&p_full, j & 1, &abort_flag)) break;
      if (!mbar_wait(&v_full[s], (j >> 1) & 1, &abort_flag)) break;
      tc_fence_after();
      const uint64_t dv0 = desc_sw128(smem_u32(sV + s * kTaTile)), dv1 = desc_sw128(smem_u32(sV + s * kTaTile + kTaTile / 2));
#pragma unroll
      for (int k = 0; k < 4; ++k) mma_f16(tmem + 256, dp0 + 2 * k, dv0 + 2 * k, idesc, (j > 0 || k > 0) ? 1u : 0u);
#pragma unroll
      for (int k = 0; k < 4; ++k) mma_f16(tmem + 256, dp1 + 2 * k, dv1 + 2 * k, idesc, 1u);
      mma_commit(&v_empty[s]);
      mma_commit(&pv_done);
    }
  } else if (warp >= 4) {
    // ---- softmax: thread = query row of the tile = TMEM lane
    const int wq = warp & 3, row = wq * 32 + lane;
    const uint32_t tb = tmem + ((uint32_t)(wq * 32) << 16);
    // the row's prefix position (masked: its block's; clean: its own slot); rows past the data or the length see nothing
    const int pos = masked ? n0 + row / d : n0 + row;
    const bool live = row < rows && pos < S;
    const float c = a.scale_log2e;
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; j < n_kt; ++j) {
      const int s = j & 1;
      const bool own = masked && j == n_kt - 1;
      // visible key columns of this tile for this row: [lo, hi]
      int lo = 0, hi = -1;
      if (live) {
        if (own) { lo = shift + (row / d) * d; hi = shift + row; }
        else hi = min(127, pos - j * 128);
      }
      if (!mbar_wait(&s_full[s], (j >> 1) & 1, &abort_flag)) { ok = false; break; }
      tc_fence_after();
      float sv[128];
#pragma unroll
      for (int cb = 0; cb < 128; cb += 16) {
        uint32_t r[16];
        tmem_ld16(tb + s * 128 + cb, r);
        tmem_ld_wait();
#pragma unroll
        for (int q = 0; q < 16; ++q) sv[cb + q] = __uint_as_float(r[q]);
      }
      tc_fence_before();
      mbar_arrive(&s_empty[s]);
      float mt = -INFINITY;
#pragma unroll
      for (int q = 0; q < 128; ++q) {
        sv[q] = (q >= lo && q <= hi) ? sv[q] * c : -INFINITY;
        mt = fmaxf(mt, sv[q]);
      }
      float alpha = 1.f;
      if (mt > m_ref + 8.f) {               // also the first visible tile (m_ref = -inf)
        alpha = m_ref == -INFINITY ? 1.f : exp2f(m_ref - mt);
        m_ref = mt;
        l *= alpha;
      }
      const float m_use = m_ref == -INFINITY ? 0.f : m_ref;
      float lsum = 0.f;
#pragma unroll
      for (int q = 0; q < 128; ++q) {
        sv[q] = exp2f(sv[q] - m_use);       // exp2(-inf) = 0 for the hidden columns
        lsum += sv[q];
      }
      l += lsum;
      if (j > 0) {
        if (!mbar_wait(&pv_done, (j - 1) & 1, &abort_flag)) { ok = false; break; }
        tc_fence_after();
        if (__any_sync(0xffffffffu, alpha != 1.f)) {   // rescale this warp's O rows in tensor memory
#pragma unroll 1
          for (int cb = 0; cb < 128; cb += 16) {
            uint32_t r[16];
            tmem_ld16(tb + 256 + cb, r);
            tmem_ld_wait();
#pragma unroll
            for (int q = 0; q < 16; ++q) r[q] = __float_as_uint(__uint_as_float(r[q]) * alpha);
            tmem_st16(tb + 256 + cb, r);
          }
          tmem_st_wait();
        }
      }
      // P as the A operand of the second MMA: [128 rows][128 keys] in two 64-key halves, rows of 128 bytes,
      // 16-byte chunk ch of row r stored at chunk ch ^ (r & 7) (the 128-byte swizzle)
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        uint8_t* prow = sP + hf * (kTaTile / 2) + row * 128;
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) {
          uint32_t w[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const __nv_bfloat162 v2 = __floats2bfloat162_rn(sv[hf * 64 + ch * 8 + 2 * q], sv[hf * 64 + ch * 8 + 2 * q + 1]);
            w[q] = *reinterpret_cast<const uint32_t*>(&v2);
          }
          *reinterpret_cast<uint4*>(prow + ((ch ^ (row & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
      fence_async_smem();
      tc_fence_before();
      mbar_arrive(&p_full);
    }
    if (ok && mbar_wait(&pv_done, (n_kt - 1) & 1, &abort_flag)) {
      tc_fence_after();
      const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll 1
      for (int cb = 0; cb < 128; cb += 16) {
        uint32_t r[16];
        tmem_ld16(tb + 256 + cb, r);
        tmem_ld_wait();
        if (row < rows) {
          uint32_t w[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const __nv_bfloat162 v2 = __floats2bfloat162_rn(__uint_as_float(r[2 * q]) * inv, __uint_as_float(r[2 * q + 1]) * inv);
            w[q] = *reinterpret_cast<const uint32_t*>(&v2);
          }
          uint4* dst = reinterpret_cast<uint4*>(out + (size_t)row * 128 + cb);
          dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
          dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 2) { tc_fence_after(); tmem_dealloc(tmem, 512); }
  if (abort_flag && threadIdx.x == 0 && a.status != nullptr) atomicExch(a.status, DEV_TIMEOUT);
}

cudaError_t launch_train_attn(const TrainAttnArgs& a, const bf16* v, bf16* vt_c, bf16* vt_m, int ldc, int ldm, cudaStream_t st) {
  cudaError_t e = allow_dynamic_smem(reinterpret_cast<const void*>(&train_attn_kernel), kTaSmem);
  if (e != cudaSuccess) return e;
  const int L = a.prompt_len * (1 + a.draft_len), ldmax = ldc > ldm ? ldc : ldm;
  train_attn_transpose_kernel<<<dim3((ldmax + 31) / 32, 2 * (128 / 32), a.B * a.Hkv), 256, 0, st>>>(v, vt_c, vt_m, L, a.prompt_len, 128, ldc, ldm);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  const int T = train_attn_positions_per_tile(a.draft_len), n_mask_tiles = (a.prompt_len + T - 1) / T;
  train_attn_kernel<<<dim3(n_mask_tiles + a.n_clean_tiles, a.Hq, a.B), kTaThreads, kTaSmem, st>>>(a);
  return cudaGetLastError();
}

}  // namespace dart
