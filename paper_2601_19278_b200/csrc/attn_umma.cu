// Split-KV grouped-query attention of the drafting step on the 5th-generation tensor cores (Section 3.1: the K
// query rows read the whole prefix and, causally, each other; Appendix B: grouped-query heads).  Same split, same
// partials and the same hi + lo operand pairs as attn_splitkv_kernel (attention.cu), whose combine kernel finishes
// both; what changes is the data path, because at batch > 1 that kernel is bound by the issue rate of its
// mma.sync pairs (tensor pipe 42 % busy at 2.1 TB/s on 16 sequences):
//   * a CTA runs two (sequence, KV head, chunk) pipelines side by side -- two consecutive chunks of one sequence,
//     which share the Q tiles -- each with its own producer thread (TMA, 128-byte swizzle, two K and two V stages
//     of 64 keys), MMA issuer thread, and four softmax warps;
//   * S = Q_hi K^T + Q_lo K^T by tcgen05.mma 64 x 64 (k = 128) into one of two tensor-memory buffers.  An M = 64
//     accumulator puts row r in lane 32 (r / 16) + r % 16, so each of the four softmax warps of a pipeline owns
//     16 rows (lanes 0..15 of its lane quarter) and all four schedulers take part;
//   * one thread per query row: exp2 against a reference maximum that only moves when exceeded by 2^8 (O rescaled
//     in tensor memory then), P split into bf16 hi + lo tiles written in the operand layout;
//   * O += P_hi V + P_lo V by tcgen05.mma 64 x 128 (k = 64) with the V tile as stored (MN-major B operand).
// The step's own K new rows are one more chunk: a 16-row side tile (rows 0..7 hi parts, 8..15 lo parts), so score
// columns c and c + 8 add up to q.k and the weight of column c is repeated on column c + 8 for v_lo.
// Every mbarrier wait is bounded; d_h = 128.
#include "common.cuh"
#include "kernels.h"
#include "umma.cuh"
#include "umma_attn.cuh"

namespace dart {

using namespace umma;

constexpr int kAuThreads = 384;                 // warps 0/2: producers, 1/3: MMA issuers, 4-7 and 8-11: softmax
constexpr int kAuQ = 64 * 128 * 2;              // 64 query rows x 128: two 64-column halves of 8 KB
constexpr int kAuP = 64 * 64 * 2;               // 64 query rows x 64 keys
constexpr int kAuKV = 64 * 128 * 2;             // 64 keys x 128: two 64-column halves
// Q hi, Q lo | P [pipeline][buffer][hi, lo] | K [pipeline][stage] | V [pipeline][stage].
constexpr size_t kAuSmem = (size_t)2 * kAuQ + 8 * kAuP + 8 * kAuKV + 1024;

__global__ void __launch_bounds__(kAuThreads, 1) attn_umma_kernel(const __grid_constant__ AttnUmmaArgs a) {
  const AttnParams& p = a.a.p;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = sm;                                    // hi, lo
  uint8_t* sP = sm + 2 * kAuQ;
  uint8_t* sK = sP + 8 * kAuP;
  uint8_t* sV = sK + 4 * kAuKV;
  __shared__ uint64_t q_full, k_full[2][2], k_empty[2][2], v_full[2][2], v_empty[2][2];
  __shared__ uint64_t s_full[2][2], s_empty[2][2], p_full[2][2], pv_done[2][2];
  __shared__ uint32_t tmem_base;
  __shared__ int abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int hk = blockIdx.y, b = blockIdx.z;
  const int P = p.seq_lens[b];          // an input of the step: readable before the previous kernel has finished
  const int n_cc = (P + p.chunk_keys - 1) / p.chunk_keys;   // cache chunks of this sequence; chunk n_cc = the new rows
  const int ci0 = 2 * (int)blockIdx.x;
  if (ci0 > n_cc) return;
  const int n_pl = ci0 + 1 <= n_cc ? 2 : 1;
  const int G = p.Hq / p.Hkv, R = G * p.K;

  if (threadIdx.x == 0) {
    mbar_init(&q_full, 1);
    for (int pl = 0; pl < 2; ++pl)
      for (int s = 0; s < 2; ++s) {
        mbar_init(&k_full[pl][s], 1); mbar_init(&k_empty[pl][s], 1); mbar_init(&v_full[pl][s], 1); mbar_init(&v_empty[pl][s], 1);
        mbar_init(&s_full[pl][s], 1); mbar_init(&s_empty[pl][s], 4);     // one arrival per softmax warp
        mbar_init(&p_full[pl][s], 4); mbar_init(&pv_done[pl][s], 1);
      }
    abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 2) tmem_alloc(&tmem_base, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base;      // pipeline pl: columns 256 pl + {0, 64}: two S buffers; 256 pl + 128: O

  // the pipeline this warp serves and its chunk
  const int pl = warp < 4 ? warp >> 1 : (warp - 4) >> 2;
  const int ci = ci0 + pl;
  const bool is_new = ci == n_cc;
  const int k_begin = is_new ? 0 : ci * p.chunk_keys;
  const int k_end = is_new ? 16 : min(P, k_begin + p.chunk_keys);
  const int n_t = (k_end - k_begin + 63) >> 6;
  const bool pl_on = pl < n_pl;

  if ((warp == 0 || warp == 2) && lane == 0 && pl_on) {
    // ---- producer of pipeline pl.  Cache rows below P_b were written by earlier steps, so their first tiles are
    // requested while the QKV kernel is still finishing; q and the new rows' side tile are its outputs.
    const int row0 = is_new ? (b * p.Hkv + hk) * 16 : (int)(((long long)b * p.Hkv + hk) * p.P_cap) + k_begin;
    const CUtensorMap* mk = is_new ? &a.mapKn : &a.mapK;
    const CUtensorMap* mv = is_new ? &a.mapVn : &a.mapV;
    auto load_tile = [&](int t) {
      const int s = t & 1;
      uint8_t* kd = sK + (pl * 2 + s) * kAuKV;
      uint8_t* vd = sV + (pl * 2 + s) * kAuKV;
      mbar_expect_tx(&k_full[pl][s], kAuKV);
      tma_load_2d(kd, mk, &k_full[pl][s], 0, row0 + t * 64);
      tma_load_2d(kd + kAuKV / 2, mk, &k_full[pl][s], 64, row0 + t * 64);
      mbar_expect_tx(&v_full[pl][s], kAuKV);
      tma_load_2d(vd, mv, &v_full[pl][s], 0, row0 + t * 64);
      tma_load_2d(vd + kAuKV / 2, mv, &v_full[pl][s], 64, row0 + t * 64);
    };
    int t = 0;
    if (!is_new)
      for (; t < n_t && t < 2; ++t) load_tile(t);
    pdl_wait();
    if (pl == 0) {
      const int q_row = (b * p.Hq + hk * G) * p.K;
      mbar_expect_tx(&q_full, 2 * kAuQ);
      tma_load_2d(sQ, &a.mapQhi, &q_full, 0, q_row);
      tma_load_2d(sQ + kAuQ / 2, &a.mapQhi, &q_full, 64, q_row);
      tma_load_2d(sQ + kAuQ, &a.mapQlo, &q_full, 0, q_row);
      tma_load_2d(sQ + kAuQ + kAuQ / 2, &a.mapQlo, &q_full, 64, q_row);
    }
    for (; t < n_t; ++t) {
      const int s = t & 1;
      if (t >= 2) {
        if (!ta_wait(&k_empty[pl][s], ((t >> 1) - 1) & 1, &abort_flag)) break;
        if (!ta_wait(&v_empty[pl][s], ((t >> 1) - 1) & 1, &abort_flag)) break;
      }
      load_tile(t);
    }
  } else if ((warp == 1 || warp == 3) && lane == 0 && pl_on) {
    // ---- MMA issuer of pipeline pl
    constexpr uint32_t idesc_s = idesc_bf16(64, 64), idesc_o = idesc_bf16(64, 128) | kIdescBMnMajor;
    const uint64_t dqh0 = desc_sw128(smem_u32(sQ)), dqh1 = desc_sw128(smem_u32(sQ + kAuQ / 2));
    const uint64_t dql0 = desc_sw128(smem_u32(sQ + kAuQ)), dql1 = desc_sw128(smem_u32(sQ + kAuQ + kAuQ / 2));
    bool ok = ta_wait(&q_full, 0, &abort_flag);
    auto issue_s = [&](int t) -> bool {      // S[t & 1] = (Q_hi + Q_lo) K_t^T
      const int s = t & 1;
      if (!ta_wait(&k_full[pl][s], (t >> 1) & 1, &abort_flag)) return false;
      if (t >= 2 && !ta_wait(&s_empty[pl][s], ((t >> 1) - 1) & 1, &abort_flag)) return false;
      tc_fence_after();
      const uint64_t dk0 = desc_sw128(smem_u32(sK + (pl * 2 + s) * kAuKV)), dk1 = desc_sw128(smem_u32(sK + (pl * 2 + s) * kAuKV + kAuKV / 2));
      const uint32_t acc = tmem + pl * 256 + s * 64;
#pragma unroll
      for (int k = 0; k < 4; ++k) mma_f16(acc, dqh0 + 2 * k, dk0 + 2 * k, idesc_s, k > 0 ? 1u : 0u);
#pragma unroll
      for (int k = 0; k < 4; ++k) mma_f16(acc, dqh1 + 2 * k, dk1 + 2 * k, idesc_s, 1u);
#pragma unroll
      for (int k = 0; k < 4; ++k) mma_f16(acc, dql0 + 2 * k, dk0 + 2 * k, idesc_s, 1u);
#pragma unroll
      for (int k = 0; k < 4; ++k) mma_f16(acc, dql1 + 2 * k, dk1 + 2 * k, idesc_s, 1u);
      mma_commit(&s_full[pl][s]);
      mma_commit(&k_empty[pl][s]);
      return true;
    };
    if (ok) ok = issue_s(0);
    for (int t = 0; t < n_t && ok; ++t) {
      const int s = t & 1;
      if (t + 1 < n_t && !issue_s(t + 1)) break;
      if (!ta_wait(&v_full[pl][s], (t >> 1) & 1, &abort_flag)) break;
      if (!ta_wait(&p_full[pl][s], (t >> 1) & 1, &abort_flag)) break;
      tc_fence_after();
      const uint64_t dv = desc_sw128_mn(smem_u32(sV + (pl * 2 + s) * kAuKV), kAuKV / 2);
      const uint64_t dph = desc_sw128(smem_u32(sP + ((pl * 2 + s) * 2) * kAuP)), dpl = desc_sw128(smem_u32(sP + ((pl * 2 + s) * 2 + 1) * kAuP));
#pragma unroll
      for (int k = 0; k < 4; ++k) mma_f16(tmem + pl * 256 + 128, dph + 2 * k, dv + 128 * k, idesc_o, (t > 0 || k > 0) ? 1u : 0u);
#pragma unroll
      for (int k = 0; k < 4; ++k) mma_f16(tmem + pl * 256 + 128, dpl + 2 * k, dv + 128 * k, idesc_o, 1u);
      mma_commit(&pv_done[pl][s]);
      mma_commit(&v_empty[pl][s]);
    }
  } else if (warp >= 4 && pl_on) {
    // ---- softmax of pipeline pl: lanes 0..15 of warp quarter wq own query rows 16 wq .. 16 wq + 15 (the M = 64
    // accumulator layout); lanes 16..31 only take part in the warp-wide tensor-memory instructions
    const int wq = warp & 3;
    const bool act = lane < 16;
    const int row = act ? wq * 16 + lane : 64;
    const uint32_t tb = tmem + ((uint32_t)(wq * 32) << 16) + pl * 256;
    const int r = row % p.K;             // position of the row inside its sequence's K-block
    const float c = rsqrtf(128.f) * 1.4426950408889634f;   // 1/sqrt(d_h) * log2(e)
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    for (int t = 0; t < n_t; ++t) {
      const int s = t & 1;
      if (!ta_wait(&s_full[pl][s], (t >> 1) & 1, &abort_flag)) { ok = false; break; }
      tc_fence_after();
      float sv[64];
      tmem_ld64(tb + s * 64, sv);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&s_empty[pl][s]);
      if (is_new) {      // columns c and c + 8 hold q.k_hi and q.k_lo of new row c; row r reads new rows c <= r
#pragma unroll
        for (int q = 0; q < 8; ++q) sv[q] = (q < p.K && q <= r) ? sv[q] + sv[q + 8] : -INFINITY;
#pragma unroll
        for (int q = 8; q < 64; ++q) sv[q] = -INFINITY;
      } else if (k_begin + t * 64 + 64 > k_end) {   // the chunk's last tile: keys past its end are hidden
        const int hi = k_end - (k_begin + t * 64) - 1;
#pragma unroll
        for (int q = 0; q < 64; ++q) sv[q] = q <= hi ? sv[q] : -INFINITY;
      }
      float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int q = 0; q < 64; ++q) mx[q & 3] = fmaxf(mx[q & 3], sv[q]);
      const float mt = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * c;
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
      if (is_new) {
#pragma unroll
        for (int q = 0; q < 8; ++q) sv[q + 8] = sv[q];   // the same weights on the v_lo rows (not part of the sum)
      }
      // keys past the chunk's end (and the rows after the 16 of the new-rows tile) have weight 0, but whatever the
      // cache holds there -- possibly not even a number -- would still enter 0 * v: those V rows are zeroed
      const int valid = is_new ? 16 : min(64, k_end - (k_begin + t * 64));
      if (valid < 64) {
        if (!ta_wait(&v_full[pl][s], (t >> 1) & 1, &abort_flag)) { ok = false; break; }
        if (act && row >= valid) {
          uint8_t* vrow = sV + (pl * 2 + s) * kAuKV + row * 128;
#pragma unroll
          for (int ch = 0; ch < 8; ++ch) {
            *reinterpret_cast<uint4*>(vrow + ch * 16) = make_uint4(0u, 0u, 0u, 0u);
            *reinterpret_cast<uint4*>(vrow + kAuKV / 2 + ch * 16) = make_uint4(0u, 0u, 0u, 0u);
          }
        }
      }
      // this P buffer was last read by the MMAs of tile t - 2
      if (t >= 2 && !ta_wait(&pv_done[pl][s], ((t >> 1) - 1) & 1, &abort_flag)) { ok = false; break; }
      if (t > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {   // rescale this warp's O rows in tensor memory
        if (!ta_wait(&pv_done[pl][s ^ 1], ((t - 1) >> 1) & 1, &abort_flag)) { ok = false; break; }   // O holds tiles 0..t-1
        tc_fence_after();
#pragma unroll 1
        for (int cb = 0; cb < 128; cb += 16) {
          uint32_t rr[16];
          tmem_ld16(tb + 128 + cb, rr);
          tmem_ld_wait();
#pragma unroll
          for (int q = 0; q < 16; ++q) rr[q] = __float_as_uint(__uint_as_float(rr[q]) * alpha);
          tmem_st16(tb + 128 + cb, rr);
        }
        tmem_st_wait();
      }
      // P as hi + lo A operands: [64 rows][64 keys] each, rows of 128 bytes, 16-byte chunk ch of row r stored at
      // chunk ch ^ (r & 7) (the 128-byte swizzle)
      uint8_t* ph = sP + ((pl * 2 + s) * 2) * kAuP + (row & 63) * 128;
      uint8_t* plo = ph + kAuP;
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) {
        if (!act) break;
        uint32_t wh[4], wl[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float x0 = sv[ch * 8 + 2 * q], x1 = sv[ch * 8 + 2 * q + 1];
          const __nv_bfloat162 h2 = __floats2bfloat162_rn(x0, x1);
          const __nv_bfloat162 l2 = __floats2bfloat162_rn(x0 - __low2float(h2), x1 - __high2float(h2));
          wh[q] = *reinterpret_cast<const uint32_t*>(&h2);
          wl[q] = *reinterpret_cast<const uint32_t*>(&l2);
        }
        const int off = (ch ^ (row & 7)) << 4;
        *reinterpret_cast<uint4*>(ph + off) = make_uint4(wh[0], wh[1], wh[2], wh[3]);
        *reinterpret_cast<uint4*>(plo + off) = make_uint4(wl[0], wl[1], wl[2], wl[3]);
      }
      fence_async_smem();
      tc_fence_before();
      __syncwarp();                          // every lane's P chunks and fences precede the warp's one arrival
      if (lane == 0) mbar_arrive(&p_full[pl][s]);
    }
    if (ok && ta_wait(&pv_done[pl][(n_t - 1) & 1], ((n_t - 1) >> 1) & 1, &abort_flag)) {
      tc_fence_after();
      // the chunk's partial: (reference maximum, sum, un-normalised output), merged by attn_combine_kernel
      const size_t slot = ((size_t)(a.a.chunk_base[b] + ci) * p.Hkv + hk) * 64 + row;
#pragma unroll 1
      for (int cb = 0; cb < 128; cb += 16) {
        uint32_t rr[16];
        tmem_ld16(tb + 128 + cb, rr);
        tmem_ld_wait();
        if (act && row < R) {
          float4* dst = reinterpret_cast<float4*>(p.o_part + slot * 128 + cb);
#pragma unroll
          for (int q = 0; q < 4; ++q)
            dst[q] = make_float4(__uint_as_float(rr[4 * q]), __uint_as_float(rr[4 * q + 1]), __uint_as_float(rr[4 * q + 2]), __uint_as_float(rr[4 * q + 3]));
        }
      }
      if (act && row < R) *reinterpret_cast<float2*>(p.ml_part + slot * 2) = make_float2(m_ref, l);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 2) { tc_fence_after(); tmem_dealloc(tmem, 512); }
  if (abort_flag && threadIdx.x == 0 && a.status != nullptr) atomicExch(a.status, DEV_TIMEOUT);
}

cudaError_t attn_umma_setup() {
  return cudaFuncSetAttribute(attn_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAuSmem);
}

cudaError_t launch_attn_umma_split(const AttnUmmaArgs& a, int max_chunks, cudaStream_t st) {
  const AttnParams& p = a.a.p;
  return launch_pdl(attn_umma_kernel, dim3((max_chunks + 1) / 2, p.Hkv, p.B), dim3(kAuThreads), kAuSmem, st, a);
}

}  // namespace dart
