// Finalize kernels: sum the split partials of a projection in a fixed order and apply the
// element-wise / row-wise op that follows it in the draft layer (Section 3.2):
//   stage_inputs : z = [RMSNorm(g) ; RMSNorm(e)], residual = g     (g = FC(features) or <mask>)
//   qkv_finalize : RoPE on q, k at position P_b + r; write q and the new rows' k, v as hi/lo pairs,
//                  append the fresh rows' k, v to the cache
//   res_norm     : x = residual + proj ; n = RMSNorm(x)             (after o_proj and after down)
//   gate_up      : u = SiLU(gate) * up
// Outputs that feed the next projection are written as bf16 hi + lo pairs.
#include "common.cuh"
#include "kernels.h"

namespace dart {

__device__ __forceinline__ float part_sum(const PartView& v, int tile, int row, int tok) {
  float s = 0.f;
  const int lo = v.clo[tile], hi = v.chi[tile];
  for (int c = lo; c <= hi; ++c) {
    const int first = (int)((((long long)c * v.U) / v.G) / v.SK);
    s += v.part[(((size_t)c * v.slots + (tile - first)) * 128 + row) * v.MP + tok];
  }
  return s;
}

__global__ void __launch_bounds__(256) stage_inputs_kernel(const StageParams p) {
  __shared__ float sh[32];
  const int m = blockIdx.x, b = m / p.K, r = m % p.K, h = p.h;
  const bool fresh = r < p.F;
  const int ftok = b * p.F + r;
  const bf16* erow = fresh ? p.embed + (size_t)min(max(p.tokens[ftok], 0), p.vocab - 1) * h : p.mask_vec + h;
  float ssg = 0.f, sse = 0.f;
  for (int n = threadIdx.x; n < h; n += blockDim.x) {
    const float g = fresh ? part_sum(p.fc, n >> 7, n & 127, ftok) : __bfloat162float(p.mask_vec[n]);
    const float e = __bfloat162float(erow[n]);
    p.res[(size_t)m * h + n] = g;
    ssg += g * g;
    sse += e * e;
  }
  ssg = block_sum(ssg, sh);
  sse = block_sum(sse, sh);
  const float rg = 1.f / sqrtf(ssg / (float)h + p.eps), re = 1.f / sqrtf(sse / (float)h + p.eps);
  for (int n = threadIdx.x; n < h; n += blockDim.x) {
    const float g = p.res[(size_t)m * h + n] * rg * __bfloat162float(p.norm_g[n]);
    const float e = __bfloat162float(erow[n]) * re * __bfloat162float(p.norm_e[n]);
    bf16 hi, lo;
    split_bf16(g, hi, lo);
    p.z_hi[(size_t)m * 2 * h + n] = hi;
    p.z_lo[(size_t)m * 2 * h + n] = lo;
    split_bf16(e, hi, lo);
    p.z_hi[(size_t)m * 2 * h + h + n] = hi;
    p.z_lo[(size_t)m * 2 * h + h + n] = lo;
  }
}

cudaError_t launch_stage_inputs(const StageParams& p, cudaStream_t st) {
  stage_inputs_kernel<<<p.B * p.K, 256, 0, st>>>(p);
  return cudaGetLastError();
}

__global__ void qkv_finalize_kernel(const QkvParams p) {
  const int m = blockIdx.x, b = m / p.K, r = m % p.K, hs = blockIdx.y, i = threadIdx.x, dh = p.dh, half = dh >> 1;
  int tile0, n0, kind;  // kind 0 q, 1 k, 2 v
  if (hs < p.Hq) { kind = 0; tile0 = p.q_tile0; n0 = hs * dh; }
  else if (hs < p.Hq + p.Hkv) { kind = 1; tile0 = p.k_tile0; n0 = (hs - p.Hq) * dh; }
  else { kind = 2; tile0 = p.v_tile0; n0 = (hs - p.Hq - p.Hkv) * dh; }
  const int na = n0 + i, nb = n0 + i + half;
  const float x1 = part_sum(p.qkv, tile0 + (na >> 7), na & 127, m);
  const float x2 = part_sum(p.qkv, tile0 + (nb >> 7), nb & 127, m);
  const long long pos = (long long)p.seq_lens[b] + r;
  float o1 = x1, o2 = x2;
  if (kind < 2) {
    const double inv = pow((double)p.rope_theta, -2.0 * (double)i / (double)dh);
    double sn, cs;
    sincos((double)pos * inv, &sn, &cs);
    o1 = (float)((double)x1 * cs - (double)x2 * sn);
    o2 = (float)((double)x2 * cs + (double)x1 * sn);
  }
  bf16 h1, l1, h2, l2;
  split_bf16(o1, h1, l1);
  split_bf16(o2, h2, l2);
  if (kind == 0) {
    const size_t o = (((size_t)b * p.Hq + hs) * p.K + r) * dh;
    p.q_hi[o + i] = h1; p.q_hi[o + i + half] = h2;
    p.q_lo[o + i] = l1; p.q_lo[o + i + half] = l2;
  } else {
    const int hk = (kind == 1) ? hs - p.Hq : hs - p.Hq - p.Hkv;
    bf16* side = (kind == 1 ? p.k_new : p.v_new) + ((size_t)b * p.Hkv + hk) * 16 * dh;
    side[(size_t)r * dh + i] = h1; side[(size_t)r * dh + i + half] = h2;
    side[(size_t)(8 + r) * dh + i] = l1; side[(size_t)(8 + r) * dh + i + half] = l2;
    if (r < p.F) {  // a fresh position: its k, v become part of the prefix cache
      bf16* dst = (kind == 1 ? p.k_cache : p.v_cache) + (((size_t)b * p.Hkv + hk) * p.P_cap + pos) * dh;
      dst[i] = h1;
      dst[i + half] = h2;
    }
  }
}

cudaError_t launch_qkv_finalize(const QkvParams& p, cudaStream_t st) {
  dim3 grid(p.B * p.K, p.Hq + 2 * p.Hkv);
  qkv_finalize_kernel<<<grid, p.dh / 2, 0, st>>>(p);
  return cudaGetLastError();
}

__global__ void __launch_bounds__(256) res_norm_kernel(const ResNormParams p) {
  __shared__ float sh[32];
  const int m = blockIdx.x, h = p.h;
  float ss = 0.f;
  for (int n = threadIdx.x; n < h; n += blockDim.x) {
    const float x = p.res[(size_t)m * h + n] + part_sum(p.proj, n >> 7, n & 127, m);
    p.res[(size_t)m * h + n] = x;
    ss += x * x;
  }
  ss = block_sum(ss, sh);
  const float rs = 1.f / sqrtf(ss / (float)h + p.eps);
  for (int n = threadIdx.x; n < h; n += blockDim.x) {
    const float v = p.res[(size_t)m * h + n] * rs * __bfloat162float(p.gamma[n]);
    bf16 hi, lo;
    split_bf16(v, hi, lo);
    p.n_hi[(size_t)m * h + n] = hi;
    p.n_lo[(size_t)m * h + n] = lo;
  }
}

cudaError_t launch_res_norm(const ResNormParams& p, cudaStream_t st) {
  res_norm_kernel<<<p.M, 256, 0, st>>>(p);
  return cudaGetLastError();
}

__global__ void __launch_bounds__(256) gate_up_kernel(const GateUpParams p) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x, m = blockIdx.y;
  if (n >= p.I) return;
  const float gt = part_sum(p.gu, n >> 7, n & 127, m);
  const float up = part_sum(p.gu, p.up_tile0 + (n >> 7), n & 127, m);
  const float u = gt / (1.f + expf(-gt)) * up;
  bf16 hi, lo;
  split_bf16(u, hi, lo);
  p.u_hi[(size_t)m * p.I + n] = hi;
  p.u_lo[(size_t)m * p.I + n] = lo;
}

cudaError_t launch_gate_up(const GateUpParams& p, cudaStream_t st) {
  dim3 grid((p.I + 255) / 256, p.M);
  gate_up_kernel<<<grid, 256, 0, st>>>(p);
  return cudaGetLastError();
}

}  // namespace dart
