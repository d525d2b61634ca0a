// The gate / up projection with row ownership (Section 3.2's SiLU-gated MLP): u = SiLU(rstd * W_gate n) * (rstd * W_up n).
//
// umma_gemm.cu balances the SMs by cutting the (tile, k-block) space into equal ranges, which splits every output
// tile between CTAs: pieces in global memory, tickets, and a fused finalize on the kernel's tail by whichever CTA
// arrives last (3.5 - 5.5 us per projection, on the critical path of the step).  Here the OUTPUT ROWS are cut instead:
// CTA c owns rows [c * rows / G, (c + 1) * rows / G) of both matrices -- 117 or 118 of 17408 at the 14B shape -- and
// streams them over the whole reduction length: every CTA reads the same number of bytes AND holds complete results,
// so the epilogue goes from tensor memory straight to the down projection's input, with no piece, no ticket and no
// second CTA involved.  A TMA box may be any number of rows high: a stage of the ring holds the CTA's R rows x 64 k of
// W_gate, the same of W_up, and ONE activation slice; gate and up advance together, each into accumulators of its
// own, and tcgen05.mma runs with M = 128 over a tile whose rows past R are whatever shared memory holds there --
// accumulator rows that nothing reads.
// Why gate and up share a stage.  A stage of the ring costs the same ~650 cycles whatever it holds (cycle counters: the
// MMA-issuing thread spends ~370 cycles per stage on the fence, four MMAs and the commit and ~270 waiting for the
// stage; the producer ~220 on the expect-tx and two TMA issues and ~360 waiting for a free stage; the period equals
// the sum of the two issue times, with 4 stages in the ring as with 27, with or without the activation loads, with one
// commit per stage or per four).  The first form of this kernel streamed gate, then up, 118 rows x 64 k per stage:
// 22 bytes per clock, just an SM's share of HBM (gate / up stage 71.7 -> 65.6 us at the 14B shape).  With both boxes
// in a stage it is 30 KB per ~770 cycles (61.6 us; 45.1 -> 41.5 us at the 8B shape, whose 83 rows per SM were too few
// to stream alone).  And at 33 .. 128 token rows, where the activation slice (32 KB) is twice a weight tile and the
// stream-K kernel, which fetches it once per 128 weight rows, is bound by the L2 -> SM path (3 bytes per weight
// byte), the slice is fetched once per two weight boxes: 2 bytes per weight byte (111 -> 86 us at 16 x 8 token rows).
// Why only gate / up: FC, o_proj and down would own 35 rows per CTA at the 14B shape and stream at 10 bytes per clock
// (95 / 39 / 104 us instead of 41 / 25 / 43: measured), so they stay on the stream-K kernel, whose stages hold 128 rows.
// Shapes: MP = 8, 32 or 128 token rows (accumulators of 2 MP columns: column 2 t is token t's hi part, 2 t + 1 its lo
// part); up to 128 weight rows per CTA and matrix, or -- MP <= 32 -- up to 256 as two halves of 128 with an accumulator
// each (a 32B-shaped MLP is 173 rows per SM; the second half's MMAs read 16 KB further into the weight box).
// Roles, barriers, bounded waits and programmatic dependent launch are those of umma_gemm.cu.
#include "common.cuh"
#include "kernels.h"
#include "umma.cuh"

namespace dart {

using namespace umma;

constexpr int kOwnThreads = 256;
constexpr size_t kOwnSmemLimit = 220 * 1024;

template <int MP, int H>
__global__ void __launch_bounds__(kOwnThreads, 1) umma_own_kernel(const __grid_constant__ OwnArgs a) {
  constexpr int N = 2 * MP, XB = N * 64 * 2, TC = 2 * H * N;      // accumulator columns, bytes of a slice, tensor-memory columns
  static_assert(TC == 32 || TC == 64 || TC == 128 || TC == 256 || TC == 512, "tensor-memory columns: a power of two");
  extern __shared__ uint8_t smem_raw[];
  uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ uint64_t full[8], empty[8], acc_full;
  __shared__ uint32_t tmem_base;
  __shared__ int abort_flag, s_bad;
  __shared__ float s_rstd[MP];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int c = blockIdx.x, G = gridDim.x;
  const int r0 = (int)(((long long)c * a.rows) / G), r1 = (int)(((long long)(c + 1) * a.rows) / G);
  const int stages = a.stages, stage_bytes = a.stage_bytes, w_area = (stage_bytes - XB) / 2;   // [gate | up | x]
  const int KB = a.KB;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(&acc_full, 1);
    abort_flag = 0;
    s_bad = 0;
    fence_barrier_init();
    // this thread is the producer: the weights of the first stages are requested before anything else of the set-up
    const int pre = KB < stages ? KB : stages;
    const uint64_t wpol = l2_policy_evict_first();
    for (int it = 0; it < pre; ++it) {
      uint8_t* st = ring + (size_t)it * stage_bytes;
      mbar_expect_tx(&full[it], 2 * a.w_tx_bytes + XB);
      tma_load_2d_hint(st, &a.mapW[0], &full[it], it * 64, r0, wpol);
      tma_load_2d_hint(st + w_area, &a.mapW[1], &full[it], it * 64, r0, wpol);
    }
  }
  if (warp == 2) tmem_alloc(&tmem_base, TC);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base;

  if (warp == 0 && lane == 0) {
    // ---- producer: activations depend on the previous kernel
    const int pre = KB < stages ? KB : stages;
    const uint64_t wpol = l2_policy_evict_first();
    pdl_wait();
    for (int it = 0; it < pre; ++it)
      tma_load_3d(ring + (size_t)it * stage_bytes + 2 * w_area, &a.mapX, &full[it], it * 64, 0, 0);
    int s = pre == stages ? 0 : pre, ph = pre == stages ? 1 : 0;
    for (int kb = pre; kb < KB; ++kb) {
      if (!mbar_wait(&empty[s], (ph - 1) & 1, &abort_flag)) break;
      uint8_t* st = ring + (size_t)s * stage_bytes;
      mbar_expect_tx(&full[s], 2 * a.w_tx_bytes + XB);
      tma_load_2d_hint(st, &a.mapW[0], &full[s], kb * 64, r0, wpol);
      tma_load_2d_hint(st + w_area, &a.mapW[1], &full[s], kb * 64, r0, wpol);
      tma_load_3d(st + 2 * w_area, &a.mapX, &full[s], kb * 64, 0, 0);
      if (++s == stages) { s = 0; ++ph; }
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer: accumulator (matrix g, row half hh) at tensor-memory columns (g H + hh) N
    constexpr uint32_t idesc = idesc_bf16(128, N);
    int s = 0, ph = 0;
    bool ok = true;
    for (int kb = 0; kb < KB; ++kb) {
      if (!mbar_wait(&full[s], ph & 1, &abort_flag)) { ok = false; break; }
      tc_fence_after();
      const uint32_t wa = smem_u32(ring + (size_t)s * stage_bytes);
      const uint64_t xd = desc_sw128(wa + 2 * w_area);
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int g = 0; g < 2; ++g)
#pragma unroll
          for (int hh = 0; hh < H; ++hh)      // rows 128 hh .. of the box: 16 KB further on
            mma_f16(tmem + (g * H + hh) * N, desc_sw128(wa + g * w_area + hh * 16384) + 2 * k, xd + 2 * k, idesc, (kb > 0 || k > 0) ? 1u : 0u);
      mma_commit(&empty[s]);
      if (++s == stages) { s = 0; ++ph; }
    }
    if (ok) mma_commit(&acc_full);
  } else if (warp >= 4) {
    // ---- epilogue: one output row per thread and row half (row = tensor-memory lane), eight tokens at a time
    const int wq = warp & 3, M = a.M;
    pdl_wait();   // the sums of squares below are the previous kernel's; u may still be read by the one before it
    for (int t = wq * (MP / 4); t < (wq + 1) * (MP / 4); ++t) {     // 1/rms of this projection's input, a quarter of the tokens per warp
      float sacc = 0.f;
      if (t < M)
        for (int tl = lane; tl < a.ss_tiles; tl += 32) sacc += __ldcg(a.ss_in + (size_t)tl * a.ss_mp + t);
      sacc = warp_sum(sacc);
      if (lane == 0) s_rstd[t] = t < M ? 1.f / sqrtf(sacc / (float)a.h + a.eps) : 0.f;
    }
    if (!mbar_wait_relaxed(&acc_full, 0, &abort_flag)) s_bad = 1;
    asm volatile("bar.sync 1, 128;" ::: "memory");   // s_rstd is written; the four warps agree on what follows
    if (!s_bad) {
      tc_fence_after();
      const uint32_t tbase = tmem + ((uint32_t)(wq * 32) << 16);
#pragma unroll 1
      for (int hh = 0; hh < H; ++hh) {
        const int row = hh * 128 + wq * 32 + lane, n = r0 + row;
        const bool has_row = row < r1 - r0;
#pragma unroll 1
        for (int ch = 0; ch < MP / 8 && ch * 8 < M; ++ch) {
          uint32_t rg[16], ru[16];
          tmem_ld16(tbase + hh * N + 16 * ch, rg);
          tmem_ld16(tbase + (H + hh) * N + 16 * ch, ru);
          tmem_ld_wait();
          if (has_row) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int t = ch * 8 + j;
              if (t < M) {
                const float gt = s_rstd[t] * (__uint_as_float(rg[2 * j]) + __uint_as_float(rg[2 * j + 1]));
                const float up = s_rstd[t] * (__uint_as_float(ru[2 * j]) + __uint_as_float(ru[2 * j + 1]));
                bf16 hi, lo;
                split_bf16(gt / (1.f + expf(-gt)) * up, hi, lo);
                DART_CHECK(n < a.rows && n < a.ld_out, a.status) {
                  a.out_hi[(size_t)t * a.ld_out + n] = hi;
                  a.out_lo[(size_t)t * a.ld_out + n] = lo;
                }
              }
            }
          }
        }
      }
    }
  }
  pdl_wait();
  pdl_trigger();
  tc_fence_before();
  __syncthreads();
  if (warp == 2) { tc_fence_after(); tmem_dealloc(tmem, TC); }
  if (abort_flag && threadIdx.x == 0) {
    atomicExch(a.status, DEV_TIMEOUT);
    for (int i = 0; i < 100; ++i) __nanosleep(1000);
  }
}

// Plan of the kernel above for MP = 8, 32 or 128 token rows: at least kOwnMinRows / 2 rows per CTA and matrix (two
// boxes to a stage: enough bytes to stream), at most 128 (MP = 128) or 256; two to eight stages.
bool own_plan_make(OwnPlan* p, int rows, int Kd, int n_sm, int MP) {
  p->rows = rows; p->Kd = Kd; p->KB = (Kd + 63) / 64;
  p->grid = rows < n_sm ? rows : n_sm;
  p->R = (rows + p->grid - 1) / p->grid;
  if (p->R < kOwnMinRows / 2 || p->R > (MP == 128 ? 128 : 256)) return false;
  const int H = p->R > 128 ? 2 : 1, xb = 2 * MP * 128;
  const int w_area = ((p->R + 7) / 8) * 8 * 128;
  p->stage_bytes = 2 * w_area + xb;
  p->w_tx_bytes = p->R * 128;
  // the MMAs read H x 128 rows from a weight box's base: past gate's rows they read up's, past up's the activation
  // slice and, in the ring's last stage, this much beyond it
  int tail = H * 16384 - w_area - xb;
  tail = tail > 0 ? ((tail + 1023) / 1024) * 1024 : 0;
  int stages = (int)((kOwnSmemLimit - 1024 - tail) / p->stage_bytes);
  if (stages > 8) stages = 8;
  if (stages < 2) return false;
  p->stages = stages;
  p->smem = (size_t)stages * p->stage_bytes + tail + 1024;
  return true;
}

template <int MP, int H>
static cudaError_t launch_own_t(const OwnPlan& plan, const OwnArgs& a, cudaStream_t st) {
  const cudaError_t e = allow_dynamic_smem(reinterpret_cast<const void*>(umma_own_kernel<MP, H>), kOwnSmemLimit);
  if (e != cudaSuccess) return e;
  return launch_pdl(umma_own_kernel<MP, H>, dim3(plan.grid), dim3(kOwnThreads), plan.smem, st, a);
}

cudaError_t launch_umma_own(const OwnPlan& plan, const CUtensorMap* mapW, const CUtensorMap& mapX, int M, const EpiArgs& epi,
                                 int* status, cudaStream_t st) {
  OwnArgs a;
  memset(&a, 0, sizeof(a));
  a.mapW[0] = mapW[0]; a.mapW[1] = mapW[1];
  a.mapX = mapX;
  a.rows = plan.rows; a.KB = plan.KB; a.M = M;
  a.stages = plan.stages; a.stage_bytes = plan.stage_bytes; a.w_tx_bytes = plan.w_tx_bytes;
  a.ss_in = epi.ss_in; a.ss_tiles = epi.ss_tiles; a.ss_mp = epi.ss_mp; a.h = epi.h; a.eps = epi.eps;
  a.out_hi = epi.out_hi; a.out_lo = epi.out_lo; a.ld_out = epi.ld_out;
  a.status = status;
  const int MP = padded_tokens(M);
  if (MP == 128) return launch_own_t<128, 1>(plan, a, st);
  if (MP == 32) return plan.R > 128 ? launch_own_t<32, 2>(plan, a, st) : launch_own_t<32, 1>(plan, a, st);
  if (MP == 8) return plan.R > 128 ? launch_own_t<8, 2>(plan, a, st) : launch_own_t<8, 1>(plan, a, st);
  return cudaErrorInvalidValue;
}

}  // namespace dart
