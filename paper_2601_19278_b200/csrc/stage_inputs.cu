// Small kernels that stage the inputs of the draft layer (Section 3.2): the <mask> rows' z row and its 1/rms
// (constants of the model, written once at init), the RoPE (cos, sin) table, the copy of the <mask> row into the z
// rows of a batch, and -- when the caller passes pre-fused features g -- what the feature FC's prologue and
// epilogue would have written.
#include "common.cuh"
#include "kernels.h"
#include "finalize.cuh"

namespace dart {

// The <mask> rows are the same for every sequence and every step: their z row ([m_g * gain_g (not yet
// normalised) ; RMSNorm(m_e)]) and the 1/rms of m_g are computed once, at init.
__global__ void __launch_bounds__(256) mask_row_kernel(const bf16* mask_vec, const bf16* norm_g, const bf16* norm_e, int h,
                                                       float eps, bf16* z_hi, bf16* z_lo, float* rstd_mask, float* mask_res) {
  __shared__ float sh[32];
  float sg = 0.f, se = 0.f;
  for (int n = threadIdx.x; n < h; n += blockDim.x) {
    const float g = __bfloat162float(mask_vec[n]), e = __bfloat162float(mask_vec[h + n]);
    sg += g * g;
    se += e * e;
  }
  sg = block_sum(sg, sh);
  se = block_sum(se, sh);
  const float re = 1.f / sqrtf(se / (float)h + eps);
  if (threadIdx.x == 0) rstd_mask[0] = 1.f / sqrtf(sg / (float)h + eps);
  for (int n = threadIdx.x; n < h; n += blockDim.x) {
    bf16 hi, lo;
    split_bf16(__bfloat162float(mask_vec[n]) * __bfloat162float(norm_g[n]), hi, lo);
    z_hi[n] = hi; z_lo[n] = lo;
    mask_res[n] = __bfloat162float(mask_vec[n]);
    split_bf16(__bfloat162float(mask_vec[h + n]) * re * __bfloat162float(norm_e[n]), hi, lo);
    z_hi[h + n] = hi; z_lo[h + n] = lo;
  }
}

// (cos, sin) of every (position, frequency) pair the cache can hold, computed once in double precision.
__global__ void rope_table_kernel(float2* tab, int n_pos, int half, double theta, int dh) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)n_pos * half) return;
  const int pos = (int)(idx / half), i = (int)(idx % half);
  const double inv = pow(theta, -2.0 * (double)i / (double)dh);
  double sn, cs;
  sincos((double)pos * inv, &sn, &cs);
  tab[idx] = make_float2((float)cs, (float)sn);
}

cudaError_t launch_rope_table(float2* tab, int n_pos, int dh, float theta, cudaStream_t st) {
  const long long n = (long long)n_pos * (dh / 2);
  rope_table_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(tab, n_pos, dh / 2, (double)theta, dh);
  return cudaGetLastError();
}

__global__ void fill_mask_rows_kernel(bf16* z_hi, bf16* z_lo, const bf16* zmask_hi, const bf16* zmask_lo, int K, const FreshOffsets foff,
                                      int width) {
  const int tok = blockIdx.x, b = tok / K;
  if (tok % K < foff.v[b + 1] - foff.v[b]) return;
  const uint4* sh = reinterpret_cast<const uint4*>(zmask_hi);
  const uint4* sl = reinterpret_cast<const uint4*>(zmask_lo);
  uint4* dh = reinterpret_cast<uint4*>(z_hi + (size_t)tok * width);
  uint4* dl = reinterpret_cast<uint4*>(z_lo + (size_t)tok * width);
  for (int i = threadIdx.x; i < width / 8; i += blockDim.x) { dh[i] = sh[i]; dl[i] = sl[i]; }
}

cudaError_t launch_fill_mask_rows(bf16* z_hi, bf16* z_lo, const bf16* zmask_hi, const bf16* zmask_lo, int B, int K,
                                  const FreshOffsets& foff, int width, cudaStream_t st) {
  fill_mask_rows_kernel<<<B * K, 256, 0, st>>>(z_hi, z_lo, zmask_hi, zmask_lo, K, foff, width);
  return cudaGetLastError();
}

// Pre-fused features (feat_in = 0): the caller hands g [fresh rows][h] itself, so the feature FC is skipped and
// this kernel does what its prologue and epilogue do for one fresh row per block (Section 3.2): the residual
// g as fp32, z's g half = hi/lo of g * gain, the sums of squares of g per 128-column tile (the 1/rms is applied
// after the QKV projection), and z's e half = RMSNorm of the next token's embedding.
__global__ void __launch_bounds__(128) prefused_rows_kernel(const EpiArgs e, const bf16* __restrict__ g, int MP) {
  __shared__ float sh[32];
  const int t = blockIdx.x, tid = threadIdx.x;
  pdl_wait();
  const int orow = fresh_to_step_row(e, t);
  const bf16* grow = g + (size_t)t * e.h;
  for (int n0 = 0, tile = 0; n0 < e.h; n0 += 128, ++tile) {
    const int n = n0 + tid;
    float x = 0.f;
    if (n < e.h) {
      x = __bfloat162float(grow[n]);
      e.res0[(size_t)t * e.h + n] = x;
      bf16 hi, lo;
      split_bf16(x * __bfloat162float(e.gamma[n]), hi, lo);
      e.out_hi[(size_t)orow * e.ld_out + n] = hi;
      e.out_lo[(size_t)orow * e.ld_out + n] = lo;
    }
    const float ss = block_sum(x * x, sh);
    if (tid == 0) e.ss_out[(size_t)tile * MP + t] = ss;
  }
  // the shifted token embedding of this fresh row
  const int id = min(max(e.tokens[t], 0), e.vocab - 1);
  const bf16* row = e.embed + (size_t)id * e.h;
  float ss = 0.f;
  for (int n = tid; n < e.h; n += 128) {
    const float v = __bfloat162float(row[n]);
    ss += v * v;
  }
  ss = block_sum(ss, sh);
  const float rs = 1.f / sqrtf(ss / (float)e.h + e.eps);
  for (int n = tid; n < e.h; n += 128) {
    bf16 hi, lo;
    split_bf16(__bfloat162float(row[n]) * rs * __bfloat162float(e.gamma_e[n]), hi, lo);
    e.out_hi[(size_t)orow * e.ld_out + e.h + n] = hi;
    e.out_lo[(size_t)orow * e.ld_out + e.h + n] = lo;
  }
}

cudaError_t launch_prefused_rows(const EpiArgs& e, const bf16* g, int n_fresh, cudaStream_t st) {
  return launch_pdl(prefused_rows_kernel, dim3(n_fresh), dim3(128), 0, st, e, g, padded_tokens(n_fresh));
}

cudaError_t launch_mask_row(const bf16* mask_vec, const bf16* norm_g, const bf16* norm_e, int h, float eps, bf16* z_hi,
                            bf16* z_lo, float* rstd_mask, float* mask_res, cudaStream_t st) {
  mask_row_kernel<<<1, 256, 0, st>>>(mask_vec, norm_g, norm_e, h, eps, z_hi, z_lo, rstd_mask, mask_res);
  return cudaGetLastError();
}

}  // namespace dart
