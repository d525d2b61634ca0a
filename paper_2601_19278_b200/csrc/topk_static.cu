// dart_topk_rows_noalloc: per-row log-softmax + top-k of caller-provided logits, for callers that must
// not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need candidates: a serving
// process that handed all of HBM to its own pool at start-up, a latency-critical loop where an allocation
// (an implicit device synchronisation) is forbidden, or a plug-in that runs under somebody else's
// memory budget and has no handle of ours to hold a workspace.  For them this entry point needs no
// dart_handle and no workspace: its scratch is a fixed array that lives in the library's own device image.
//
// The computation is the two-phase selection that dart_draft_step performs after its LM head
// (Algorithm 1 lines 6-8 at temperature 0): phase 1 cuts every row into kSlices vocabulary slices and
// writes each slice's (max, sum-exp) and best `topk` entries to the scratch; phase 2 is the library's
// ordinary merge kernel reading that scratch.
//
// The scratch is one array per GPU, shared by every call and never cleared: phase 1 overwrites exactly
// the entries phase 2 reads, so nothing has to start at zero, but two calls that overlap on the same GPU
// (different streams, or different host threads) race on it.
#include <stdint.h>
#include <string.h>

#include "../../include/dart.h"
#include "common.cuh"
#include "kernels.h"

namespace dart {

constexpr int kMaxRows = 128;  // largest `rows` a call may pass
constexpr int kSlices = 32;    // vocabulary slices per row = CTAs per row in phase 1
// per (slice, row): 2 floats of statistics + 32 keys + 32 logits + 32 ids
constexpr size_t kScratchFloats = (size_t)kSlices * kMaxRows * (2 + 3 * 32);

// 1.6 MB that every GPU which loads the library holds until the process exits.
static __device__ __align__(256) float g_topk_scratch[kScratchFloats];

// In host code `g_topk_scratch` is only a stand-in symbol, not a device address: the address is
// obtained once per device with cudaGetSymbolAddress and cached here.
static float* g_scratch_ptr[64] = {nullptr};

__device__ __forceinline__ void slice_list_insert(float& lk, int& lid, float nk, int nid, int lane) {
  const bool before = (lk > nk) || (lk == nk && lid < nid);
  const int pos = __popc(__ballot_sync(0xffffffffu, before));
  const float pk = __shfl_up_sync(0xffffffffu, lk, 1);
  const int pid = __shfl_up_sync(0xffffffffu, lid, 1);
  if (lane == pos) { lk = nk; lid = nid; }
  else if (lane > pos) { lk = pk; lid = pid; }
}

// Phase 1: block (slice, row) scans logits[row][v0..v1): max, sum-exp, best `topk` (value desc, id asc).
__global__ void __launch_bounds__(256) slice_partials_kernel(const float* logits, int vocab, int MP, int topk, float* stats,
                                                             float* keys, float* ys, int32_t* ids) {
  __shared__ float sh[32];
  __shared__ float wk[8][32];
  __shared__ int wi[8][32];
  const int c = blockIdx.x, tk = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int v0 = (int)(((long long)c * vocab) / kSlices), v1 = (int)(((long long)(c + 1) * vocab) / kSlices);
  const float* row = logits + (size_t)tk * vocab;

  float mx = -INFINITY;
  for (int v = v0 + tid; v < v1; v += 256) mx = fmaxf(mx, row[v]);
  mx = warp_max(mx);
  if (lane == 0) sh[warp] = mx;
  __syncthreads();
  mx = sh[0];
  for (int i = 1; i < 8; ++i) mx = fmaxf(mx, sh[i]);
  float sum = 0.f;
  for (int v = v0 + tid; v < v1; v += 256) sum += expf(row[v] - mx);
  sum = block_sum(sum, sh);

  // every warp keeps the best 32 of its strided share, one entry per lane
  float lk = -INFINITY;
  int lid = 0x7fffffff;
  for (int base = v0 + warp * 32; base < v1; base += 256) {
    const int v = base + lane;
    const bool ok = v < v1;
    const float key = ok ? row[v] : -INFINITY;
    float thr = __shfl_sync(0xffffffffu, lk, topk - 1);
    unsigned mask = __ballot_sync(0xffffffffu, ok && key > thr);
    while (mask) {
      const int src = __ffs(mask) - 1;
      slice_list_insert(lk, lid, __shfl_sync(0xffffffffu, key, src), base + src, lane);
      thr = __shfl_sync(0xffffffffu, lk, topk - 1);
      mask &= mask - 1;
      mask &= __ballot_sync(0xffffffffu, ok && key > thr);
    }
  }
  wk[warp][lane] = lk;
  wi[warp][lane] = lid;
  __syncthreads();
  if (warp == 0) {
    for (int w = 1; w < 8; ++w) {
      const float key = wk[w][lane];
      const int id = wi[w][lane];
      const bool ok = lane < topk && key > -INFINITY;
      float tkv = __shfl_sync(0xffffffffu, lk, topk - 1);
      int tiv = __shfl_sync(0xffffffffu, lid, topk - 1);
      unsigned mask = __ballot_sync(0xffffffffu, ok && (key > tkv || (key == tkv && id < tiv)));
      while (mask) {
        const int src = __ffs(mask) - 1;
        slice_list_insert(lk, lid, __shfl_sync(0xffffffffu, key, src), __shfl_sync(0xffffffffu, id, src), lane);
        tkv = __shfl_sync(0xffffffffu, lk, topk - 1);
        tiv = __shfl_sync(0xffffffffu, lid, topk - 1);
        mask &= mask - 1;
        mask &= __ballot_sync(0xffffffffu, ok && (key > tkv || (key == tkv && id < tiv)));
      }
    }
    const size_t o = ((size_t)c * MP + tk) * 32 + lane;
    keys[o] = lk;
    ys[o] = lk;       // temperature 0: the selection key is the logit itself
    ids[o] = lid;
    if (lane == 0) {
      stats[((size_t)c * MP + tk) * 2] = mx;
      stats[((size_t)c * MP + tk) * 2 + 1] = sum;
    }
  }
}

}  // namespace dart

using namespace dart;

extern "C" int dart_topk_rows_noalloc(const float* logits, int32_t rows, int32_t vocab, int32_t topk, float eps_logit,
                                      int32_t* out_ids, float* out_slogit, void* cuda_stream) {
  if (logits == nullptr || out_ids == nullptr || out_slogit == nullptr) return DART_ERR_INVALID_ARG;
  if (rows < 1 || vocab < 1 || topk < 1 || topk > 32 || topk > vocab || !(eps_logit >= 0.f)) return DART_ERR_INVALID_ARG;
  if (rows > kMaxRows) return DART_ERR_CAPACITY;  // the static scratch holds at most kMaxRows rows
  int dev = 0, major = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) { record_global_cuda_error(e); return DART_ERR_CUDA; }
  if (dev < 0 || dev >= 64) return DART_ERR_INVALID_ARG;   // the address cache below holds 64 devices
  if (g_scratch_ptr[dev] == nullptr) {
    // first call on this device (it must be the current device): check the architecture once and resolve the
    // array's device address.  Two host threads that get here together both store the same address: benign.
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) { record_global_cuda_error(e); return DART_ERR_CUDA; }
    if (major != 10) return DART_ERR_UNSUPPORTED_ARCH;
    float* ptr = nullptr;
    e = cudaGetSymbolAddress((void**)&ptr, g_topk_scratch);
    if (e != cudaSuccess || ptr == nullptr) { record_global_cuda_error(e); return DART_ERR_CUDA; }
    g_scratch_ptr[dev] = ptr;
  }
  float* base = g_scratch_ptr[dev];
  const int MP = padded_tokens(rows);
  LmParams p;
  memset(&p, 0, sizeof(p));
  p.M = rows; p.V = vocab; p.topk = topk; p.eps_logit = eps_logit; p.grid = kSlices;
  p.part_stats = base;
  p.part_key = base + (size_t)kSlices * kMaxRows * 2;
  p.part_y = p.part_key + (size_t)kSlices * kMaxRows * 32;
  p.part_id = reinterpret_cast<int32_t*>(p.part_y + (size_t)kSlices * kMaxRows * 32);
  p.out_ids = out_ids; p.out_slogit = out_slogit;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  slice_partials_kernel<<<dim3(kSlices, rows), 256, 0, st>>>(logits, vocab, MP, topk, p.part_stats, p.part_key, p.part_y, p.part_id);
  if ((e = cudaGetLastError()) != cudaSuccess) { record_global_cuda_error(e); return DART_ERR_CUDA; }
  if ((e = launch_topk_merge(p, st)) != cudaSuccess) { record_global_cuda_error(e); return DART_ERR_CUDA; }
  return DART_OK;
}
