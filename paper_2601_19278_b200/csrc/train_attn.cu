// Forward attention under the prefix-shared training mask (Section 3.3, Appendix B): a packed row of
// `prompt_len` clean positions followed by one block of `draft_len` masked positions per prefix position; block n
// reads prompt slots 0..n and, causally, itself; clean positions read causally.  The mask is block-sparse with a
// regular structure, so no mask tensor exists: a CTA owns 128 query rows --
//   * a clean tile: 128 consecutive prompt slots, or
//   * a masked tile: the blocks of T = 128 / draft_len consecutive prefix positions (T * draft_len <= 128 rows) --
// of TWO query heads that share a KV head (grouped-query attention: one K / V^T tile in shared memory serves both,
// which halves the L2 -> SM traffic per flop; with one head per CTA the kernel was bound by it), and walks exactly
// the 64-key tiles its rows can see: the clean key tiles up to its last prefix position (only those that reach past
// its first position need a per-row bound) and, for a masked tile, its own slots (same block and causal).
// Flash-attention dataflow on the 5th-generation tensor cores, per head, in steps of 128 keys:
//   S = Q K^T       tcgen05.mma (128 x 128, k = 128), operands by TMA (128-byte swizzle), one S buffer in tensor memory
//   P = exp2(S - m) four warps per head, one query row per thread, 64 key columns at a time (the S buffer is free again
//                   once its second half is in registers); bf16 P written to shared memory in the operand layout
//   O += P V        tcgen05.mma (128 x 128, k = 64) per half; V tiles are used as stored ([keys][d_h]: the MN-major form
//                   of the B operand), so no transposed copy of V exists; O stays in tensor memory
// Why 128 keys per score MMA: an MMA instruction of this shape family costs ~88 cycles of the tensor pipe whether it
// is 64 or 128 columns wide (cycle counters), so 64-key score tiles paid 8 + 4 instructions per head and 64 keys
// (0.44 of the bf16 peak on visible pairs); 128-key ones pay 4 + 4.
// The reference maximum m only moves when a tile's maximum exceeds it by more than 2^8, so the O rows are rescaled
// in tensor memory a few times per row instead of once per tile.  The two heads' softmax groups and the single MMA
// issuer run concurrently: one head's exponentials overlap the other's MMAs.  Every mbarrier wait is bounded.
#include "common.cuh"
#include "kernels.h"
#include "umma.cuh"
#include "umma_attn.cuh"

namespace dart {

using namespace umma;

constexpr int kTaThreads = 384;                         // producer, MMA issuer, TMEM owner, idle; 4 + 4 softmax warps
constexpr int kTaQ = 128 * 128 * 2;                     // a head's Q tile: two 64-column halves
constexpr int kTaKV = 128 * 128 * 2;                    // 128 keys x 128: two halves of 128 keys x 64 columns, for K and for V
constexpr int kTaP = 128 * 64 * 2;                      // a head's P tile of 64 keys (two per step)
constexpr int kTaVh = 64 * 128 * 2;                     // V of 64 keys: two halves of 64 keys x 64 columns
// Q [2 heads] | P [2 heads][2 halves] | K [2 stages of 128 keys] | V [2 stages of 64 keys, the halves of a step]: 225 KB
constexpr size_t kTaSmem = (size_t)2 * kTaQ + 4 * kTaP + 2 * kTaKV + 2 * kTaVh + 1024;

__global__ void __launch_bounds__(kTaThreads, 1) train_attn_kernel(const __grid_constant__ TrainAttnArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = sm;                                   // [2 heads]
  uint8_t* sP = sm + 2 * kTaQ;                        // [2 heads][2 halves of a step]
  uint8_t* sK = sP + 4 * kTaP;                        // [2 stages]
  uint8_t* sV = sK + 2 * kTaKV;                       // [2 halves of a step]
  __shared__ uint64_t q_full, k_full[2], k_empty[2], v_full[2], v_empty[2];
  __shared__ uint64_t s_full[2], s_empty[2], p_full[2][2], pv_done[2][2];
  __shared__ uint32_t tmem_base;
  __shared__ int abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = a.Hq / a.Hkv, pairs = (G + 1) / 2;    // query heads per KV head; CTAs (pairs of heads) per KV head
  const int b = blockIdx.z, hk = (int)blockIdx.y / pairs, hq0 = hk * G + ((int)blockIdx.y % pairs) * 2;
  const int nh = hq0 + 1 < (hk + 1) * G ? 2 : 1;      // an odd group's last CTA has one head
  const int Lp = a.prompt_len, d = a.draft_len, L = Lp * (1 + d), T = train_attn_positions_per_tile(d);
  const int n_mask_tiles = (Lp + T - 1) / T, S = a.seq_len[b];
  // heavy tiles first: masked tiles from the last prefix position down, then clean tiles from the last down
  const bool masked = (int)blockIdx.x < n_mask_tiles;
  const int ti = masked ? n_mask_tiles - 1 - (int)blockIdx.x : a.n_clean_tiles - 1 - ((int)blockIdx.x - n_mask_tiles);
  const int n0 = masked ? ti * T : ti * 128;                       // first prefix position / prompt slot of the tile
  const int q_slot0 = masked ? Lp + n0 * d : n0;                   // first packed slot of the tile's query rows
  const int rows = masked ? min(T, Lp - n0) * d : min(128, Lp - n0);
  const int last_pos = masked ? min(n0 + T, Lp) - 1 : min(n0 + 128, Lp) - 1;
  const int n_clean = n0 < S ? min(last_pos, S - 1) / 128 + 1 : 0;  // clean 128-key steps some valid row can see
  const int n_st = n0 < S ? n_clean + (masked ? 1 : 0) : 0;         // + one step over the tile's own 128 slots
  const int n_kt = 2 * n_st;                                        // 64-key halves, the softmax's unit

  if (n_kt == 0) {   // every row lies past the sequence's length: zero rows, nothing to read
    for (int h = 0; h < nh; ++h) {
      bf16* out = a.out + ((size_t)(b * a.Hq + hq0 + h) * L + q_slot0) * 128;
      for (int e = threadIdx.x; e < rows * 16; e += kTaThreads) reinterpret_cast<uint4*>(out)[e] = make_uint4(0u, 0u, 0u, 0u);
    }
    return;
  }
  if (threadIdx.x == 0) {
    mbar_init(&q_full, 1);
    for (int s = 0; s < 2; ++s) { mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], nh); }   // one release per head
    for (int s = 0; s < 2; ++s) { mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], nh); }
    for (int h = 0; h < 2; ++h) {
      mbar_init(&s_full[h], 1); mbar_init(&s_empty[h], 4);             // one arrival per softmax warp
      for (int s = 0; s < 2; ++s) { mbar_init(&p_full[h][s], 4); mbar_init(&pv_done[h][s], 1); }
    }
    abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 2) tmem_alloc(&tmem_base, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base;          // head h: columns 256 h + 0..127: S; 256 h + 128..255: O

  if (warp == 0 && lane == 0) {
    // ---- producer: the heads' Q tiles once, then per key tile K and V, [64 keys][128] each
    mbar_expect_tx(&q_full, nh * kTaQ);
    for (int h = 0; h < nh; ++h) {
      const int q_row = (b * a.Hq + hq0 + h) * L + q_slot0;
      tma_load_2d(sQ + h * kTaQ, &a.mapQ, &q_full, 0, q_row);
      tma_load_2d(sQ + h * kTaQ + kTaQ / 2, &a.mapQ, &q_full, 64, q_row);
    }
    for (int j = 0; j < n_st; ++j) {
      const int k_row = (b * a.Hkv + hk) * L + (j >= n_clean ? q_slot0 : j * 128);   // first key's packed slot
      const int st = j & 1;
      if (j >= 2 && !ta_wait(&k_empty[st], ((j >> 1) - 1) & 1, &abort_flag)) break;
      mbar_expect_tx(&k_full[st], kTaKV);
      tma_load_2d(sK + st * kTaKV, &a.mapK, &k_full[st], 0, k_row);
      tma_load_2d(sK + st * kTaKV + kTaKV / 2, &a.mapK, &k_full[st], 64, k_row);
    }
  } else if (warp == 2 && lane == 0) {
    // ---- producer of the V tiles, 64 keys at a time: the half of a step's keys whose P V product is done is
    // replaced at once (with V in whole steps and one stage, the MMA threads waited for V a fifth of the time).  A
    // thread of its own: a V stage comes free much later than a K stage, and behind it in one queue the K loads
    // would start that much later too.
    for (int t = 0; t < n_kt; ++t) {
      const int j = t >> 1, hf = t & 1;
      const int k_row = (b * a.Hkv + hk) * L + (j >= n_clean ? q_slot0 : j * 128) + 64 * hf;
      if (t >= 2 && !ta_wait(&v_empty[hf], (j - 1) & 1, &abort_flag)) break;
      mbar_expect_tx(&v_full[hf], kTaVh);
      tma_load_2d(sV + hf * kTaVh, &a.mapV, &v_full[hf], 0, k_row);
      tma_load_2d(sV + hf * kTaVh + kTaVh / 2, &a.mapV, &v_full[hf], 64, k_row);
    }
  } else if ((warp == 1 || warp == 3) && lane == 0 && (warp >> 1) < nh) {
    // ---- MMA issuer of head h (the two heads are independent pipelines that share the K / V^T stages)
    const int h = warp >> 1;
    constexpr uint32_t idesc_s = idesc_bf16(128, 128), idesc_o = idesc_bf16(128, 128);
    const uint64_t dq0 = desc_sw128(smem_u32(sQ + h * kTaQ)), dq1 = desc_sw128(smem_u32(sQ + h * kTaQ + kTaQ / 2));
    bool ok = ta_wait(&q_full, 0, &abort_flag);
    auto issue_s = [&](int j) -> bool {      // S = Q K_j^T over the step's 128 keys
      const int st = j & 1;
      if (!ta_wait(&k_full[st], (j >> 1) & 1, &abort_flag)) return false;
      if (j >= 1 && !ta_wait(&s_empty[h], (j - 1) & 1, &abort_flag)) return false;
      tc_fence_after();
      const uint64_t dk0 = desc_sw128(smem_u32(sK + st * kTaKV)), dk1 = desc_sw128(smem_u32(sK + st * kTaKV + kTaKV / 2));
      const uint32_t acc = tmem + h * 256;
#pragma unroll
      for (int k = 0; k < 4; ++k) mma_f16(acc, dq0 + 2 * k, dk0 + 2 * k, idesc_s, k > 0 ? 1u : 0u);
#pragma unroll
      for (int k = 0; k < 4; ++k) mma_f16(acc, dq1 + 2 * k, dk1 + 2 * k, idesc_s, 1u);
      mma_commit(&s_full[h]);
      mma_commit(&k_empty[st]);
      return true;
    };
    if (ok) ok = issue_s(0);
    // V as stored ([keys][d_h], d_h contiguous) is the MN-major form of the B operand: 8-key groups 1024 bytes
    // apart, the two 64-wide halves of d_h kTaVh / 2 bytes apart, the 16 keys of one MMA 2048 bytes on
    for (int j = 0; j < n_st && ok; ++j) {
      for (int hf = 0; hf < 2 && ok; ++hf) {
        if (!ta_wait(&v_full[hf], j & 1, &abort_flag)) { ok = false; break; }
        if (!ta_wait(&p_full[h][hf], j & 1, &abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint64_t dp = desc_sw128(smem_u32(sP + (h * 2 + hf) * kTaP));
        const uint64_t dv = desc_sw128_mn(smem_u32(sV + hf * kTaVh), kTaVh / 2);
#pragma unroll
        for (int k = 0; k < 4; ++k)
          mma_f16(tmem + h * 256 + 128, dp + 2 * k, dv + 128 * k, idesc_o | kIdescBMnMajor, (j > 0 || hf > 0 || k > 0) ? 1u : 0u);
        mma_commit(&pv_done[h][hf]);
        mma_commit(&v_empty[hf]);
        // the next step's scores between the two halves: its S buffer came free when the softmax took the second
        // half of this step's scores into registers
        if (hf == 0 && j + 1 < n_st && !issue_s(j + 1)) ok = false;
      }
    }
  } else if (warp >= 4 && (warp - 4) / 4 < nh) {
    // ---- softmax of head h: thread = query row of the tile = TMEM lane
    const int h = (warp - 4) / 4, wq = warp & 3, row = wq * 32 + lane;
    const uint32_t tb = tmem + ((uint32_t)(wq * 32) << 16) + h * 256;
    // the row's prefix position (masked: its block's; clean: its own slot); rows past the data or the length give zeros
    const int pos = masked ? n0 + row / d : n0 + row;
    const bool live = row < rows && pos < S;
    const float c = a.scale_log2e;
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; j < n_kt; ++j) {      // j: 64-key half (j & 1) of step j >> 1
      const int sb = j & 1;
      const bool own = j >= 2 * n_clean;
      // visible key columns of this tile for this row: [lo, hi]; tiles below the tile's first position need no bound
      const bool bounded = own || j * 64 + 63 > n0;
      int lo = 0, hi = 63;
      if (own) { lo = (row / d) * d - (j - 2 * n_clean) * 64; hi = row - (j - 2 * n_clean) * 64; }
      else if (bounded) hi = pos - j * 64;
      if (sb == 0 && !ta_wait(&s_full[h], (j >> 1) & 1, &abort_flag)) { ok = false; break; }
      tc_fence_after();
      float sv[64];
      tmem_ld64(tb + sb * 64, sv);
      if (sb == 1) {                         // both halves of the step's scores are in registers: the buffer is free
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&s_empty[h]);
      }
      if (bounded) {
#pragma unroll
        for (int q = 0; q < 64; ++q) sv[q] = (q >= lo && q <= hi) ? sv[q] : -INFINITY;
      }
      float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four chains instead of one of 64 dependent maxima
#pragma unroll
      for (int q = 0; q < 64; ++q) mx[q & 3] = fmaxf(mx[q & 3], sv[q]);
      const float mt = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * c;      // c > 0: the scaled maximum
      float alpha = 1.f;
      if (mt > m_ref + 8.f) {               // also the first visible tile (m_ref = -inf)
        alpha = m_ref == -INFINITY ? 1.f : ex2(m_ref - mt);
        m_ref = mt;
        l *= alpha;
      }
      const float m_use = m_ref == -INFINITY ? 0.f : m_ref;
      float ls[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int q = 0; q < 64; ++q) {
        sv[q] = ex2(fmaf(sv[q], c, -m_use));   // ex2(-inf) = 0 for the hidden columns
        ls[q & 3] += sv[q];
      }
      l += (ls[0] + ls[1]) + (ls[2] + ls[3]);
      const int pb = j & 1;
      // this P buffer was last read by the MMA of tile j - 2
      if (j >= 2 && !ta_wait(&pv_done[h][pb], ((j >> 1) - 1) & 1, &abort_flag)) { ok = false; break; }
      if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {   // rescale this warp's O rows in tensor memory
        if (!ta_wait(&pv_done[h][pb ^ 1], ((j - 1) >> 1) & 1, &abort_flag)) { ok = false; break; }   // O holds tiles 0..j-1
        tc_fence_after();
        {
#pragma unroll 1
          for (int cb = 0; cb < 128; cb += 16) {
            uint32_t r[16];
            tmem_ld16(tb + 128 + cb, r);
            tmem_ld_wait();
#pragma unroll
            for (int q = 0; q < 16; ++q) r[q] = __float_as_uint(__uint_as_float(r[q]) * alpha);
            tmem_st16(tb + 128 + cb, r);
          }
          tmem_st_wait();
        }
      }
      uint8_t* prow = sP + (h * 2 + pb) * kTaP + row * 128;
      // P as the A operand of the second MMA: [128 rows][64 keys], rows of 128 bytes, 16-byte chunk ch of row r
      // stored at chunk ch ^ (r & 7) (the 128-byte swizzle)
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) {
        uint32_t w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const __nv_bfloat162 v2 = __floats2bfloat162_rn(sv[ch * 8 + 2 * q], sv[ch * 8 + 2 * q + 1]);
          w[q] = *reinterpret_cast<const uint32_t*>(&v2);
        }
        *reinterpret_cast<uint4*>(prow + ((ch ^ (row & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
      }
      fence_async_smem();
      tc_fence_before();
      __syncwarp();                          // every lane's P chunks and fences precede the warp's one arrival
      if (lane == 0) mbar_arrive(&p_full[h][pb]);
    }
    if (ok && ta_wait(&pv_done[h][(n_kt - 1) & 1], ((n_kt - 1) >> 1) & 1, &abort_flag)) {
      tc_fence_after();
      const float inv = (live && l > 0.f) ? 1.f / l : 0.f;
      bf16* out = a.out + ((size_t)(b * a.Hq + hq0 + h) * L + q_slot0) * 128;
#pragma unroll 1
      for (int cb = 0; cb < 128; cb += 16) {
        uint32_t r[16];
        tmem_ld16(tb + 128 + cb, r);
        tmem_ld_wait();
        if (row < rows) {
          uint32_t w[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const float x0 = live ? __uint_as_float(r[2 * q]) * inv : 0.f, x1 = live ? __uint_as_float(r[2 * q + 1]) * inv : 0.f;
            const __nv_bfloat162 v2 = __floats2bfloat162_rn(x0, x1);
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

cudaError_t launch_train_attn(const TrainAttnArgs& a, cudaStream_t st) {
  cudaError_t e = allow_dynamic_smem(reinterpret_cast<const void*>(&train_attn_kernel), kTaSmem);
  if (e != cudaSuccess) return e;
  const int T = train_attn_positions_per_tile(a.draft_len), n_mask_tiles = (a.prompt_len + T - 1) / T;
  const int G = a.Hq / a.Hkv;   // one CTA per pair of query heads of a KV head
  train_attn_kernel<<<dim3(n_mask_tiles + a.n_clean_tiles, a.Hkv * ((G + 1) / 2), a.B), kTaThreads, kTaSmem, st>>>(a);
  return cudaGetLastError();
}

}  // namespace dart
