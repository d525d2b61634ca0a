// Split-KV grouped-query attention of the drafting step on the 5th-generation tensor cores (Section 3.1: the K
// query rows read the whole prefix and, causally, each other; Appendix B: grouped-query heads).  Same split, same
// partials and the same hi + lo operand pairs as attn_splitkv_kernel (attention.cu), whose combine kernel finishes
// both; what changes is the data path, because at batch > 1 that kernel is bound by the issue rate of its
// mma.sync pairs (tensor pipe 42 % busy at 2.1 TB/s on 16 sequences):
//   * a CTA runs two (sequence, KV head, chunk) pipelines side by side -- two consecutive chunks of one sequence,
//     which share the Q tile -- each with its own producer thread (TMA, 128-byte swizzle, three K and two V stages
//     of 64 keys, loaded independently: a K stage is free once its scores are in tensor memory, a full tile earlier
//     than the V stage of the same keys, and its refill has to cover the HBM latency before the next-but-one score
//     MMA), MMA issuer thread, and four softmax warps;
//   * the hi and lo parts of an operand are stacked along M: rows 32 q + i of the 128-row Q tile hold Q_hi of query
//     row 16 q + i, rows 32 q + 16 + i hold Q_lo of the same row (i < 16, q = warp quarter), so ONE tcgen05.mma
//     128 x 64 (k = 128) leaves q_hi.k in tensor-memory lane 32 q + i and q_lo.k in lane 32 q + 16 + i: the two
//     lanes belong to the same warp, and the score is their sum, exchanged by shuffles.  (The cost of an MMA here
//     hardly depends on M, so stacking halves the tensor time against one MMA per part.)
//   * two threads per query row: lane i of a warp takes key columns 0..31, lane 16 + i columns 32..63 (after the
//     exchange each holds the full score of its columns); exp2 against a reference maximum shared by the pair that
//     only moves when exceeded by 2^8 (O rescaled in tensor memory then); P is written as bf16 hi and lo rows of
//     one 128-row operand tile laid out like Q;
//   * O_hi / O_lo += P V by ONE tcgen05.mma 128 x 128 (k = 64) with the V tile as stored (MN-major B operand); the
//     two accumulator rows of a query row are added once, when the chunk's partial is written.
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
constexpr int kAuQ = 128 * 128 * 2;             // 128 operand rows (hi and lo of 64 query rows) x 128: two 64-column halves
constexpr int kAuP = 128 * 64 * 2;              // 128 operand rows (hi and lo of 64 query rows) x 64 keys
constexpr int kAuKV = 64 * 128 * 2;             // 64 keys x 128: two 64-column halves
constexpr int kAuKStages = 3, kAuVStages = 2;
// Q | P [pipeline] | K [pipeline][stage] | V [pipeline][stage].  One P tile per pipeline is enough: the MMAs that
// read it finish a few hundred cycles after it is complete, long before the next tile's weights exist.
constexpr size_t kAuSmem = (size_t)kAuQ + 2 * kAuP + 2 * (kAuKStages + kAuVStages) * kAuKV + 1024;

__global__ void __launch_bounds__(kAuThreads, 1) attn_umma_kernel(const __grid_constant__ AttnUmmaArgs a) {
  const AttnParams& p = a.a.p;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = sm;
  uint8_t* sP = sm + kAuQ;
  uint8_t* sK = sP + 2 * kAuP;
  uint8_t* sV = sK + 2 * kAuKStages * kAuKV;
  __shared__ uint64_t q_full, k_full[2][kAuKStages], k_empty[2][kAuKStages], v_full[2][2], v_empty[2][2];
  __shared__ uint64_t s_full[2][2], s_empty[2][2], p_full[2], pv_done[2];
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
    for (int pl = 0; pl < 2; ++pl) {
      for (int s = 0; s < kAuKStages; ++s) { mbar_init(&k_full[pl][s], 1); mbar_init(&k_empty[pl][s], 1); }
      for (int s = 0; s < 2; ++s) {
        mbar_init(&v_full[pl][s], 1); mbar_init(&v_empty[pl][s], 1);
        mbar_init(&s_full[pl][s], 1); mbar_init(&s_empty[pl][s], 4);     // one arrival per softmax warp
      }
      mbar_init(&p_full[pl], 4); mbar_init(&pv_done[pl], 1);
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
    auto load_k = [&](int t, int s) {
      uint8_t* kd = sK + (pl * kAuKStages + s) * kAuKV;
      mbar_expect_tx(&k_full[pl][s], kAuKV);
      tma_load_2d(kd, mk, &k_full[pl][s], 0, row0 + t * 64);
      tma_load_2d(kd + kAuKV / 2, mk, &k_full[pl][s], 64, row0 + t * 64);
    };
    auto load_v = [&](int t) {
      const int s = t & 1;
      uint8_t* vd = sV + (pl * 2 + s) * kAuKV;
      mbar_expect_tx(&v_full[pl][s], kAuKV);
      tma_load_2d(vd, mv, &v_full[pl][s], 0, row0 + t * 64);
      tma_load_2d(vd + kAuKV / 2, mv, &v_full[pl][s], 64, row0 + t * 64);
    };
    // the first tiles (K 0, 1, 2 and V 0, 1) find their stages free
    if (!is_new) {
      for (int t = 0; t < n_t && t < kAuKStages; ++t) load_k(t, t);
      for (int t = 0; t < n_t && t < 2; ++t) load_v(t);
    }
    pdl_wait();
    if (pl == 0) {
      const int q_row = (b * p.Hq + hk * G) * p.K;
      mbar_expect_tx(&q_full, kAuQ);
      for (int q4 = 0; q4 < 4; ++q4)        // 16 query rows per warp quarter: hi rows, then lo rows, per 64-column half
        for (int ch = 0; ch < 2; ++ch) {
          uint8_t* d = sQ + ch * (kAuQ / 2) + q4 * 32 * 128;
          tma_load_2d(d, &a.mapQhi, &q_full, ch * 64, q_row + 16 * q4);
          tma_load_2d(d + 16 * 128, &a.mapQlo, &q_full, ch * 64, q_row + 16 * q4);
        }
    }
    if (is_new) { load_k(0, 0); load_v(0); }     // one tile, written by the QKV kernel
    // then, in the order in which the stages come free: K of tile t + 1 (after the scores of tile t - 2), V of tile t
    // (after the P V product of tile t - 2)
    int ks = 0, kph = 0;      // stage and round of K tile t + 1
    for (int t = 2; t < n_t; ++t) {
      if (t + 1 < n_t) {
        if (!ta_wait(&k_empty[pl][ks], kph & 1, &abort_flag)) break;
        load_k(t + 1, ks);
        if (++ks == kAuKStages) { ks = 0; ++kph; }
      }
      if (t < n_t) {
        if (!ta_wait(&v_empty[pl][t & 1], ((t >> 1) - 1) & 1, &abort_flag)) break;
        load_v(t);
      }
    }
  } else if ((warp == 1 || warp == 3) && lane == 0 && pl_on) {
    // ---- MMA issuer of pipeline pl
    constexpr uint32_t idesc_s = idesc_bf16(128, 64), idesc_o = idesc_bf16(128, 128) | kIdescBMnMajor;
    const uint64_t dq0 = desc_sw128(smem_u32(sQ)), dq1 = desc_sw128(smem_u32(sQ + kAuQ / 2));
    bool ok = ta_wait(&q_full, 0, &abort_flag);
    int ks = 0, kph = 0;                     // stage and round of the next K tile
    auto issue_s = [&](int t) -> bool {      // S[t & 1] = [Q_hi ; Q_lo] K_t^T
      const int s = t & 1;
      if (!ta_wait(&k_full[pl][ks], kph & 1, &abort_flag)) return false;
      if (t >= 2 && !ta_wait(&s_empty[pl][s], ((t >> 1) - 1) & 1, &abort_flag)) return false;
      tc_fence_after();
      const uint32_t ka = smem_u32(sK + (pl * kAuKStages + ks) * kAuKV);
      const uint64_t dk0 = desc_sw128(ka), dk1 = desc_sw128(ka + kAuKV / 2);
      const uint32_t acc = tmem + pl * 256 + s * 64;
#pragma unroll
      for (int k = 0; k < 4; ++k) mma_f16(acc, dq0 + 2 * k, dk0 + 2 * k, idesc_s, k > 0 ? 1u : 0u);
#pragma unroll
      for (int k = 0; k < 4; ++k) mma_f16(acc, dq1 + 2 * k, dk1 + 2 * k, idesc_s, 1u);
      mma_commit(&s_full[pl][s]);
      mma_commit(&k_empty[pl][ks]);
      if (++ks == kAuKStages) { ks = 0; ++kph; }
      return true;
    };
    if (ok) ok = issue_s(0);
    for (int t = 0; t < n_t && ok; ++t) {
      const int s = t & 1;
      if (t + 1 < n_t && !issue_s(t + 1)) break;
      if (!ta_wait(&v_full[pl][s], (t >> 1) & 1, &abort_flag)) break;
      if (!ta_wait(&p_full[pl], t & 1, &abort_flag)) break;
      tc_fence_after();
      const uint64_t dv = desc_sw128_mn(smem_u32(sV + (pl * 2 + s) * kAuKV), kAuKV / 2);
      const uint64_t dp = desc_sw128(smem_u32(sP + pl * kAuP));
#pragma unroll
      for (int k = 0; k < 4; ++k) mma_f16(tmem + pl * 256 + 128, dp + 2 * k, dv + 128 * k, idesc_o, (t > 0 || k > 0) ? 1u : 0u);
      mma_commit(&pv_done[pl]);
      mma_commit(&v_empty[pl][s]);
    }
  } else if (warp >= 4 && pl_on) {
    // ---- softmax of pipeline pl.  Warp quarter wq owns query rows 16 wq .. 16 wq + 15; lane i < 16 sits on the
    // tensor-memory lane of the row's hi part and takes key columns 0..31, lane 16 + i on the lo part's lane and
    // takes columns 32..63.
    const int wq = warp & 3, hh = lane >> 4;
    const int row = wq * 16 + (lane & 15);          // query row
    const uint32_t tb = tmem + ((uint32_t)(wq * 32) << 16) + pl * 256;
    const int r = row % p.K;             // position of the row inside its sequence's K-block
    const float c = rsqrtf(128.f) * 1.4426950408889634f;   // 1/sqrt(d_h) * log2(e)
    float m_ref = -INFINITY, l = 0.f;    // l: this thread's half of the row sum
    bool ok = true;
    for (int t = 0; t < n_t; ++t) {
      const int s = t & 1;
      if (!ta_wait(&s_full[pl][s], (t >> 1) & 1, &abort_flag)) { ok = false; break; }
      tc_fence_after();
      float raw[64];
      tmem_ld64(tb + s * 64, raw);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&s_empty[pl][s]);
      // score of this thread's 32 columns = its own part + the partner lane's part of the same columns
      float sv[32];
#pragma unroll
      for (int q = 0; q < 32; ++q) {
        const float send = hh ? raw[q] : raw[32 + q];
        const float got = __shfl_xor_sync(0xffffffffu, send, 16);
        sv[q] = (hh ? raw[32 + q] : raw[q]) + got;
      }
      const int c0 = 32 * hh;            // first key column of this thread
      if (is_new) {      // columns c and c + 8 hold q.k_hi and q.k_lo of new row c; row r reads new rows c <= r
#pragma unroll
        for (int q = 0; q < 8; ++q) sv[q] = (hh == 0 && q < p.K && q <= r) ? sv[q] + sv[q + 8] : -INFINITY;
#pragma unroll
        for (int q = 8; q < 32; ++q) sv[q] = -INFINITY;
      } else if (k_begin + t * 64 + 64 > k_end) {   // the chunk's last tile: keys past its end are hidden
        const int hi = k_end - (k_begin + t * 64) - 1 - c0;
#pragma unroll
        for (int q = 0; q < 32; ++q) sv[q] = q <= hi ? sv[q] : -INFINITY;
      }
      float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int q = 0; q < 32; ++q) mx[q & 3] = fmaxf(mx[q & 3], sv[q]);
      float mt = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
      mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 16)) * c;   // the row's maximum over both halves
      float alpha = 1.f;
      if (mt > m_ref + 8.f) {               // also the first visible tile (m_ref = -inf); the same in both lanes of a row
        alpha = m_ref == -INFINITY ? 1.f : ex2(m_ref - mt);
        m_ref = mt;
        l *= alpha;
      }
      const float m_use = m_ref == -INFINITY ? 0.f : m_ref;
      float ls[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int q = 0; q < 32; ++q) {
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
        if (hh == 0 && row >= valid) {      // 64 threads, one V row each
          uint8_t* vrow = sV + (pl * 2 + s) * kAuKV + row * 128;
#pragma unroll
          for (int ch = 0; ch < 8; ++ch) {
            *reinterpret_cast<uint4*>(vrow + ch * 16) = make_uint4(0u, 0u, 0u, 0u);
            *reinterpret_cast<uint4*>(vrow + kAuKV / 2 + ch * 16) = make_uint4(0u, 0u, 0u, 0u);
          }
        }
      }
      // the P tile was last read by the MMAs of tile t - 1, after which O holds tiles 0 .. t - 1
      if (t >= 1 && !ta_wait(&pv_done[pl], (t - 1) & 1, &abort_flag)) { ok = false; break; }
      if (t > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {   // rescale this warp's O rows (hi and lo parts) in tensor memory
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
      // P as one A operand of 128 rows x 64 keys laid out like Q: row 32 wq + i = hi parts of query row 16 wq + i,
      // row 32 wq + 16 + i = lo parts; rows of 128 bytes, 16-byte chunk ch of operand row x stored at chunk
      // ch ^ (x & 7) (the 128-byte swizzle).  This thread writes the 4 chunks of its 32 columns into both rows.
      const int xrow = wq * 32 + (lane & 15);
      uint8_t* ph = sP + pl * kAuP + xrow * 128;
      uint8_t* plo = ph + 16 * 128;
#pragma unroll
      for (int cq = 0; cq < 4; ++cq) {
        uint32_t wh[4], wl[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float x0 = sv[cq * 8 + 2 * q], x1 = sv[cq * 8 + 2 * q + 1];
          const __nv_bfloat162 h2 = __floats2bfloat162_rn(x0, x1);
          const __nv_bfloat162 l2 = __floats2bfloat162_rn(x0 - __low2float(h2), x1 - __high2float(h2));
          wh[q] = *reinterpret_cast<const uint32_t*>(&h2);
          wl[q] = *reinterpret_cast<const uint32_t*>(&l2);
        }
        const int off = ((4 * hh + cq) ^ (xrow & 7)) << 4;     // (xrow + 16) & 7 == xrow & 7
        *reinterpret_cast<uint4*>(ph + off) = make_uint4(wh[0], wh[1], wh[2], wh[3]);
        *reinterpret_cast<uint4*>(plo + off) = make_uint4(wl[0], wl[1], wl[2], wl[3]);
      }
      fence_async_smem();
      tc_fence_before();
      __syncwarp();                          // every lane's P chunks and fences precede the warp's one arrival
      if (lane == 0) mbar_arrive(&p_full[pl]);
    }
    if (ok && ta_wait(&pv_done[pl], (n_t - 1) & 1, &abort_flag)) {
      tc_fence_after();
      // the chunk's partial: (reference maximum, sum, un-normalised output), merged by attn_combine_kernel.  The
      // output row is the sum of the hi part's and the lo part's accumulator rows (this lane's and its partner's).
      const float lt = l + __shfl_xor_sync(0xffffffffu, l, 16);
      const size_t slot = ((size_t)(a.a.chunk_base[b] + ci) * p.Hkv + hk) * 64 + row;
#pragma unroll 1
      for (int cb = 0; cb < 128; cb += 16) {
        uint32_t rr[16];
        tmem_ld16(tb + 128 + cb, rr);
        tmem_ld_wait();
        float o[16];
#pragma unroll
        for (int q = 0; q < 16; ++q) o[q] = __uint_as_float(rr[q]) + __shfl_xor_sync(0xffffffffu, __uint_as_float(rr[q]), 16);
        if (row < R) {                       // each lane of the pair stores half of the 16 columns
          float4* dst = reinterpret_cast<float4*>(p.o_part + slot * 128 + cb + 8 * hh);
          dst[0] = hh ? make_float4(o[8], o[9], o[10], o[11]) : make_float4(o[0], o[1], o[2], o[3]);
          dst[1] = hh ? make_float4(o[12], o[13], o[14], o[15]) : make_float4(o[4], o[5], o[6], o[7]);
        }
      }
      if (hh == 0 && row < R) *reinterpret_cast<float2*>(p.ml_part + slot * 2) = make_float2(m_ref, lt);
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
