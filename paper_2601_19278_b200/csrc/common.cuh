// Device helpers shared by the kernels of the DART drafting step (sm_100a only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace dart {

typedef __nv_bfloat16 bf16;

// D(16x8,f32) += A(16x16,bf16,row) * B(16x8,bf16,col)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Split an fp32 activation into bf16 hi + bf16 lo (x ~= hi + lo to ~16 mantissa bits) so that
// a bf16 tensor-core product with fp32 accumulation keeps near-fp32 accuracy on the activation side.
__device__ __forceinline__ void split_bf16(float x, bf16& hi, bf16& lo) {
  hi = __float2bfloat16_rn(x);
  lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Block-wide sum with a fixed reduction order (deterministic). `sh` needs 32 floats.
__device__ __forceinline__ float block_sum(float v, float* sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) sh[warp] = v;
  __syncthreads();
  float r = 0.f;
  for (int i = 0; i < nw; ++i) r += sh[i];
  return r;
}

// Philox4x32-10 (Salmon et al., SC'11): ten rounds, Weyl-bumped key.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0);
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return c;
}

// Programmatic dependent launch.  Every kernel of the step is launched with the programmatic-stream-
// serialization attribute.  A kernel calls pdl_wait() before it touches anything an earlier kernel
// produced or may still be reading -- in the streaming kernels that is after the first weight loads have
// been issued -- and pdl_trigger() once its main work is done (before its epilogue), so that the next
// kernel's blocks are scheduled onto SMs as they drain and start their own weight stream early.
// pdl_wait() returns once the predecessor grid has completed and its writes are visible; since every
// kernel waits before it completes, completion is transitive along the stream.
// (Measured on B200: triggering at the *start* of the streaming kernels instead doubled the step time -- the
// early-launched successors crowd the running kernel -- so there the trigger comes late.  The short kernels between
// them -- attention split and combine, top-k merge, bigram sweep -- trigger right after their wait: their successors'
// launch and set-up then overlap them, 1.3 us per step.)
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Device status word values (mirrors dart_status for the device-detectable errors).
enum : int { DEV_OK = 0, DEV_TIMEOUT = -5, DEV_BAD_INDEX = -6 };

// Index checks of the debug build (-DDART_DEBUG): `DART_CHECK(cond, status) statement;` runs the statement only when
// cond holds and otherwise records DEV_BAD_INDEX in the status word (never traps, never faults); the release build
// compiles the statement alone.  The checks stand in for a memory sanitizer: they guard the stores whose indices
// come from the caller's lengths, counts and plans.
#ifdef DART_DEBUG
#define DART_CHECK(cond, status) if (!(cond)) { if ((status) != nullptr) atomicExch((status), (int)DEV_BAD_INDEX); } else
#else
#define DART_CHECK(cond, status)
#endif

}  // namespace dart
