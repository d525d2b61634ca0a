// Weight-streaming projections on the Blackwell data path (Section 3.2's single decoder layer: FC, QKV,
// o_proj, gate/up, down): y = W[rows, Kd] * x[M, Kd]^T for M = 8..128 token rows.
//
// The op is HBM-bound, so the kernel is built to keep as many weight bytes in flight as shared memory
// holds and to spend no load/store-unit work on them:
//   * one persistent CTA per SM; a ring of shared-memory stages, each a 128-row x 64-k bf16 weight tile
//     (16 KB) plus the matching 64-k slice of the activations (hi rows, then lo rows), both written by TMA
//     (cp.async.bulk.tensor, 128-byte swizzle) and signalled on an mbarrier;
//   * one thread issues tcgen05.mma (M = 128 weight rows, N = 2 * MP = hi and lo token rows, K = 16, four
//     per stage) straight from shared memory; the fp32 accumulator lives in tensor memory (two buffers, so
//     the next tile's MMAs overlap the previous tile's read-out); tcgen05.commit frees the stage;
//   * four warps read the accumulator out of tensor memory (tcgen05.ld), add the hi and lo halves and write
//     the CTA's fp32 piece of the tile;
//   * stream-K: the flattened (128-row tile, 64-k block) space is cut into gridDim.x equal ranges;
//     a CTA writes one fp32 piece per tile it touches and takes a ticket on the tile's group, and the CTA that
//     takes a group's last ticket runs the fused finalize (finalize.cuh) once it is past its streaming loop.
// TMA zero-fills what lies outside a matrix, so ragged row counts, k tails and missing token rows need no
// predicates here.
#include "common.cuh"
#include "kernels.h"
#include "umma.cuh"
#include "finalize.cuh"

namespace dart {

using namespace umma;

constexpr int kUmmaThreads = 512;
constexpr int kWBytes = 128 * 64 * 2;

template <int MP, bool ONE = (MP == 128)>      // ONE: one 64-k block per stage (a work unit is then two stages)
struct UmmaCfg {
  static constexpr int N = 2 * MP;                       // hi rows + lo rows
  static constexpr int XBytes = N * 64 * 2;
  // A stage holds kUmmaKS consecutive 64-k blocks of a tile (the weight boxes, then the activation slices): a stage
  // of the ring costs about the same ~690 cycles whatever it holds, and one block -- 16 KB of weights -- per stage is
  // just an SM's share of HBM.  The plans count their units in stages (GemmPlan::KR).
  // At 128 token rows a block pair would be a 96 KB stage, two to the ring (measured slower than four of 48 KB): there
  // a unit is SPU = 2 stages of one block each.  So it is for QKV at 32 token rows (59.7 us against 64.3 with block
  // pairs at a 32B shape, where o_proj and down gain from the pairs: 34.8 and 59.4 us against 36.9 and 63.5).
  static constexpr int KS = ONE ? 1 : kUmmaKS;            // 64-k blocks per stage
  static constexpr int SPU = kUmmaKS / KS;                // stages per work unit
  static constexpr int StageBytes = KS * (kWBytes + XBytes);
  static constexpr int Stages = MP == 8 ? 5 : (MP == 32 && ONE ? 8 : 4);
  static constexpr int TmemCols = 2 * N < 32 ? 32 : 2 * N;
  static constexpr size_t SmemBytes = (size_t)Stages * StageBytes + 1024;
};

// Position of unit u = tile * KB + kb of the launch, advanced one unit at a time (the single producer
// thread sits on the critical path of every stage, so it does no divisions in its loop).
// With paired tiles (pair_offset > 0: QKV's g- and e-halves, gate and up) the units run over the tiles in the order
// T, T + pair_offset, T + 1, T + 1 + pair_offset, ...: the two tiles of a group are streamed back to back, so a group is
// complete where its 2 * KR consecutive units end, the groups' ends are spread evenly over the CTAs and no CTA finalizes
// two groups in a row (in plain tile order every group ended in the second half of the CTAs).
__host__ __device__ inline int actual_tile(int v, int pair_offset) { return pair_offset > 0 ? (v & 1) * pair_offset + (v >> 1) : v; }
__host__ __device__ inline int group_of_unit_tile(int v, int pair_offset) { return pair_offset > 0 ? v >> 1 : v; }

struct UnitPos {
  int tile, kb, seg, row0, xoff, po;   // tile: position in unit order (see actual_tile)
  __device__ __forceinline__ void locate(const StreamArgs& a) {
    const int T = actual_tile(tile, po);
    seg = 0;
#pragma unroll
    for (int i = 1; i < 6; ++i)
      if (i < a.nseg && T >= a.seg[i].tile0) seg = i;
    row0 = (T - a.seg[seg].tile0) * 128;
    xoff = a.seg[seg].xoff;
  }
  __device__ __forceinline__ void set(const StreamArgs& a, long long u, int pair_offset) {
    po = pair_offset;
    tile = (int)(u / a.KR);
    kb = (int)(u - (long long)tile * a.KR);
    locate(a);
  }
  __device__ __forceinline__ void next(const StreamArgs& a) {
    if (++kb == a.KR) { kb = 0; ++tile; locate(a); }
  }
};
// Walks the ring stages of a range of units: SPU stages per unit, KS k-blocks per stage.
template <int SPU, int KS>
struct StagePos {
  UnitPos q;
  int sub;
  __device__ __forceinline__ void set(const StreamArgs& a, long long u, int pair_offset) { q.set(a, u, pair_offset); sub = 0; }
  __device__ __forceinline__ int k0(int j) const { return ((q.kb * SPU + sub) * KS + j) * 64; }   // first k of the stage's block j
  __device__ __forceinline__ void next(const StreamArgs& a) {
    if (++sub == SPU) { sub = 0; q.next(a); }
  }
};

template <int MP, bool ONE>
__global__ void __launch_bounds__(kUmmaThreads, 1) umma_rows_kernel(const __grid_constant__ UmmaGemmArgs a) {
  using C = UmmaCfg<MP, ONE>;
  const GemmArgs& p = a.g;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ uint64_t full[C::Stages], empty[C::Stages], acc_full[2], acc_empty[2];
  __shared__ uint32_t tmem_base;
  __shared__ int abort_flag;
  __shared__ int s_cnt[4];
  __shared__ float sh[32];
  __shared__ float s_emb[8];
  __shared__ float s_rstd[128];
  __shared__ int s_done[64];
  __shared__ int s_pos[128];
  __shared__ GroupMeta s_meta[kMetaSlots];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int c = blockIdx.x, G = gridDim.x;
  const int KB = p.s.KR;
  const long long u0 = ((long long)c * p.U) / G, u1 = ((long long)(c + 1) * p.U) / G;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::Stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 128); }
    abort_flag = 0;
    s_done[0] = 0;
    s_cnt[0] = s_cnt[1] = s_cnt[2] = s_cnt[3] = 0;
    fence_barrier_init();
    // this thread is the producer: weights do not depend on the previous kernel, so the ring is filled with
    // them before anything else of the CTA's setup
    const int n = (int)(u1 - u0) * C::SPU;           // stages of this CTA's range
    const int pre = n < C::Stages ? n : C::Stages;
    const uint64_t wpol = l2_policy_evict_first();
    StagePos<C::SPU, C::KS> q;
    if (n > 0) q.set(p.s, u0, p.pair_offset);
    for (int it = 0; it < pre; ++it, q.next(p.s)) {
      mbar_expect_tx(&full[it], C::StageBytes);
#pragma unroll
      for (int j = 0; j < C::KS; ++j)
        tma_load_2d_hint(ring + (size_t)it * C::StageBytes + j * kWBytes, &a.mapW[q.q.seg], &full[it], q.k0(j), q.q.row0, wpol);
    }
  }
  if (warp == 2) tmem_alloc(&tmem_base, C::TmemCols);
  if (p.epi.mode == EPI_QKV && threadIdx.x < p.s.M) {
    // inputs of the step and init-time constants: nothing an earlier kernel of this step writes
    s_pos[threadIdx.x] = p.epi.seq_lens[threadIdx.x / p.epi.K] + threadIdx.x % p.epi.K;
    s_rstd[threadIdx.x] = p.epi.rstd_mask[0];  // <mask> rows; fresh rows are overwritten in the finalize
  }
  int cand[kMetaSlots] = {-1, -1};  // groups whose piece tables sit in s_meta
  if (u0 < u1) {
    const int t0 = (int)(u0 / KB), t1 = (int)((u1 - 1) / KB);
    cand[0] = group_of_unit_tile(t0, p.pair_offset);
    cand[1] = group_of_unit_tile(t1, p.pair_offset);
    meta_prefetch(p, cand[0], &s_meta[0]);
    if (cand[1] != cand[0]) meta_prefetch(p, cand[1], &s_meta[1]);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base;

  if (warp == 0 && lane == 0) {
    // ---- producer (the ring already holds the first weights): activations depend on the previous kernel
    const int n = (int)(u1 - u0) * C::SPU;
    const int pre = n < C::Stages ? n : C::Stages;
    const uint64_t wpol = l2_policy_evict_first();
    StagePos<C::SPU, C::KS> q;
    pdl_wait();
    q.set(p.s, u0, p.pair_offset);
    for (int it = 0; it < pre; ++it, q.next(p.s)) {
      uint8_t* xs = ring + (size_t)it * C::StageBytes + C::KS * kWBytes;
#pragma unroll
      for (int j = 0; j < C::KS; ++j) {
        if (a.has_lo) tma_load_3d(xs + j * C::XBytes, &a.mapXhi, &full[it], q.q.xoff + q.k0(j), 0, 0);
        else tma_load_2d(xs + j * C::XBytes, &a.mapXhi, &full[it], q.q.xoff + q.k0(j), 0);
      }
    }
    int s = pre == C::Stages ? 0 : pre, ph = pre == C::Stages ? 1 : 0;
    for (int it = pre; it < n; ++it, q.next(p.s)) {
      if (!mbar_wait(&empty[s], (ph - 1) & 1, &abort_flag)) break;
      uint8_t* st = ring + (size_t)s * C::StageBytes;
      mbar_expect_tx(&full[s], C::StageBytes);
#pragma unroll
      for (int j = 0; j < C::KS; ++j) {
        const int k0 = q.k0(j);
        tma_load_2d_hint(st + j * kWBytes, &a.mapW[q.q.seg], &full[s], k0, q.q.row0, wpol);
        if (a.has_lo) tma_load_3d(st + C::KS * kWBytes + j * C::XBytes, &a.mapXhi, &full[s], q.q.xoff + k0, 0, 0);
        else tma_load_2d(st + C::KS * kWBytes + j * C::XBytes, &a.mapXhi, &full[s], q.q.xoff + k0, 0);
      }
      if (++s == C::Stages) { s = 0; ++ph; }
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer
    constexpr uint32_t idesc = idesc_bf16(128, C::N);
    const int n = (int)(u1 - u0) * C::SPU;
    int visit = -1, buf = 0, tile = -1;
    int t = (int)(u0 / KB), kb = (int)(u0 % KB), sub = 0, s = 0, ph = 0;
    bool ok = true;
    for (int it = 0; it < n && ok; ++it) {
      bool first = false;                            // first block of this visit: overwrite the accumulator
      if (t != tile) {
        if (tile >= 0) mma_commit(&acc_full[buf]);   // the previous tile's share is complete
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
      for (int j = 0; j < C::KS; ++j) {
        const uint64_t ad = desc_sw128(wa + j * kWBytes), bd = desc_sw128(wa + C::KS * kWBytes + j * C::XBytes);
#pragma unroll
        for (int k = 0; k < 4; ++k) mma_f16(tmem + buf * C::N, ad + 2 * k, bd + 2 * k, idesc, (!first || j > 0 || k > 0) ? 1u : 0u);
      }
      mma_commit(&empty[s]);
      if (++s == C::Stages) { s = 0; ++ph; }
      if (++sub == C::SPU) {
        sub = 0;
        if (++kb == KB) { kb = 0; ++t; }
      }
    }
    if (ok && tile >= 0) mma_commit(&acc_full[buf]);
  } else if (warp >= 4 && warp < 8) {
    // ---- read-out: TMEM lane = row of the tile; piece = [128 rows][MP tokens] fp32
    const int wq = warp & 3, row = wq * 32 + lane;
    int visit = 0;
    bool waited = false;
    long long u = u0;
    while (u < u1) {
      const int tile = (int)(u / KB);
      long long ue = (long long)(tile + 1) * KB;
      if (ue > u1) ue = u1;
      const int buf = visit & 1;
      if (!mbar_wait_relaxed(&acc_full[buf], (visit >> 1) & 1, &abort_flag)) break;
      tc_fence_after();
      if (!waited) { pdl_wait(); waited = true; }   // the piece area may still be read by the previous kernel
      float* dst = p.part + (((size_t)c * p.slots + visit) * 128 + row) * MP;
      const uint32_t tbase = tmem + ((uint32_t)(wq * 32) << 16) + buf * C::N;
#pragma unroll
      for (int ch = 0; ch < MP / 8; ++ch) {
        // hi + lo inputs: columns (2t, 2t+1) are token t's two parts; a plain input: column t is token t
        uint32_t r[16];
        float y[8];
        if (a.has_lo) {
          tmem_ld16(tbase + ch * 16, r);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 8; ++j) y[j] = __uint_as_float(r[2 * j]) + __uint_as_float(r[2 * j + 1]);
        } else {
          uint32_t q8[8];
          tmem_ld8(tbase + ch * 8, q8);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 8; ++j) y[j] = __uint_as_float(q8[j]);
        }
        const float4 v0 = make_float4(y[0], y[1], y[2], y[3]), v1 = make_float4(y[4], y[5], y[6], y[7]);
        reinterpret_cast<float4*>(dst + ch * 8)[0] = v0;
        reinterpret_cast<float4*>(dst + ch * 8)[1] = v1;
      }
      tc_fence_before();
      mbar_arrive(&acc_empty[buf]);
      // ticket of this (CTA, tile) visit: every thread releases its part of the piece, the last of the four
      // warps to get here counts.  No barrier: a warp that gave up on a wait must not strand the others.
      // (A warp can run at most three visits ahead of another - the accumulator buffers see to that - so four
      // counters suffice.)
      __threadfence();
      __syncwarp();
      if (lane == 0 && atomicAdd(&s_cnt[visit & 3], 1) == 3) {
        s_cnt[visit & 3] = 0;
        const int group = group_of_unit_tile(tile, p.pair_offset);
        if (atomicAdd(&p.ctr[group], 1) + 1 == p.expected[group]) {
          __threadfence();  // acquire: the other CTAs' pieces are visible to whatever follows the next barrier
          s_done[++s_done[0]] = group;
        }
      }
      ++visit;
      u = ue;
    }
  } else if (warp >= 8 && p.epi.mode == EPI_FC) {
    // ---- the warps with no part in the streaming: the fresh rows' shifted token embedding (its inputs are the
    // step's; the wait orders its stores after every earlier reader of z)
    pdl_wait();
    for (int ftok = c; ftok < p.s.M; ftok += G) embed_row_team<256, 1>(p.epi, threadIdx.x - 256, s_emb, ftok);
  }
  pdl_wait();
  pdl_trigger();
  asm volatile("cp.async.wait_all;" ::: "memory");
  __syncthreads();
  if (warp == 2) { tc_fence_after(); tmem_dealloc(tmem, C::TmemCols); }
  if (abort_flag) {
    // a wait ran out: report it, give copies that may still be in flight time to land, and leave
    if (threadIdx.x == 0) {
      atomicExch(a.status, DEV_TIMEOUT);
      for (int i = 0; i < 100; ++i) __nanosleep(1000);
    }
    __syncthreads();
    return;
  }
  // fused finalize of the groups this CTA completed (the ring is idle now)
  const int n_done = s_done[0];
  FinSmem* fs = reinterpret_cast<FinSmem*>(ring);
  for (int i = 0; i < n_done; ++i) {
    const int group = s_done[1 + i];
    int slot = group == cand[0] ? 0 : (group == cand[1] ? 1 : -1);
    if (slot < 0) {  // a range that touches more than two groups (short reductions): fetch the table now
      slot = 0;
      cand[0] = group;
      __syncthreads();
      meta_prefetch(p, group, &s_meta[0]);
      asm volatile("cp.async.wait_all;" ::: "memory");
      __syncthreads();
    }
    finalize_group<512, 0>(threadIdx.x, p, group, MP, sh, s_rstd, s_pos, &s_meta[slot], fs);
    if (threadIdx.x == 0) p.ctr[group] = 0;
    __syncthreads();
  }
}

template <int MP, bool ONE>
static cudaError_t launch_umma_t(const UmmaGemmArgs& a, int grid, cudaStream_t st) {
  using C = UmmaCfg<MP, ONE>;
  const cudaError_t e = allow_dynamic_smem(reinterpret_cast<const void*>(umma_rows_kernel<MP, ONE>), C::SmemBytes);
  if (e != cudaSuccess) return e;
  return launch_pdl(umma_rows_kernel<MP, ONE>, dim3(grid), dim3(kUmmaThreads), C::SmemBytes, st, a);
}

cudaError_t launch_umma_rows(const GemmPlan& plan, const UmmaMaps& maps, const GemmInput& in, const EpiArgs& epi, float* part,
                             int* status, cudaStream_t st) {
  UmmaGemmArgs a;
  memset(&a, 0, sizeof(a));
  GemmArgs& g = a.g;
  for (int i = 0; i < 6; ++i) g.s.seg[i] = plan.seg[i];
  g.s.nseg = plan.nseg; g.s.Kd = plan.Kd; g.s.SK = plan.SK; g.s.KR = plan.KR;
  g.s.x_hi = in.x_hi; g.s.x_lo = in.x_lo != nullptr ? in.x_lo : in.x_hi; g.s.ldx = in.ldx; g.s.M = in.M;
  g.slots = plan.slots; g.U = plan.U;
  g.part = part; g.meta = plan.d_meta; g.meta_stride = plan.meta_stride;
  g.ctr = plan.d_ctr; g.expected = plan.d_expected; g.pair_offset = plan.pair_offset;
  g.epi = epi;
  for (int i = 0; i < 6; ++i) a.mapW[i] = maps.W[i < plan.nseg ? i : 0];
  a.mapXhi = maps.Xhi; a.has_lo = in.x_lo != nullptr ? 1 : 0;
  a.status = status;
  const int MP = padded_tokens(in.M);
  if (MP == 8) return launch_umma_t<8, false>(a, plan.grid, st);
  if (MP == 32) return epi.mode == EPI_QKV ? launch_umma_t<32, true>(a, plan.grid, st) : launch_umma_t<32, false>(a, plan.grid, st);
  return launch_umma_t<128, true>(a, plan.grid, st);
}

}  // namespace dart
