// Split-KV grouped-query attention of the K query rows over the prefix KV cache and over each
// other (Section 3.1: strictly causal over the prefix and inside the masked block;
// Appendix B: grouped-query heads, post-RoPE keys in the cache).
//
// The new rows' k and v have already been written to cache rows P_b .. P_b+K-1, so a query
// row r simply reads cache positions s <= P_b + r.  One CTA handles one (sequence, KV head,
// chunk of keys); its (H_q/H_kv)*K query rows (<= 64) form up to four 16-row MMA tiles, one
// per warp.  KV tiles of 64 keys are staged in shared memory with cp.async (double buffered,
// XOR-swizzled 16-byte chunks), scores and P*V run on mma.sync with warp-level online
// softmax, and the per-chunk (max, sum, unnormalised output) partials are merged by
// attn_combine_kernel, which also emits the bf16 hi/lo activations for o_proj.
#include "common.cuh"
#include "kernels.h"

namespace dart {

struct AttnArgs {
  AttnParams p;
  int chunk_base[33];  // prefix sums of chunks per sequence
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N)); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}

// byte offset of 16-byte chunk `chunk` of row `row` in a [rows][DH] bf16 tile, XOR-swizzled
template <int DH>
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
  return (uint32_t)(row * (DH * 2) + ((chunk ^ (row & 7)) << 4));
}

template <int DH>
__global__ void __launch_bounds__(128) attn_splitkv_kernel(const AttnArgs a) {
  const AttnParams& p = a.p;
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int TILE_BYTES = 64 * DH * 2;
  constexpr int CH = DH / 8;  // 16-byte chunks per row
  unsigned char* Qs = smem;
  unsigned char* Ks = smem + TILE_BYTES;
  unsigned char* Vs = smem + 3 * TILE_BYTES;

  const int ci = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
  const int P = p.seq_lens[b];
  const int n_keys = P + p.K;
  const int k_begin = ci * p.chunk_keys;
  if (k_begin >= n_keys) return;
  const int k_end = min(n_keys, k_begin + p.chunk_keys);
  const int n_tiles = (k_end - k_begin + 63) >> 6;
  const int G = p.Hq / p.Hkv, R = G * p.K;
  const int n_mt = (R + 15) >> 4;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;

  const bf16* qsrc = p.q + ((size_t)b * p.Hq + (size_t)hk * G) * p.K * DH;
  const bf16* kbase = p.k_cache + ((size_t)b * p.Hkv + hk) * p.P_cap * DH;
  const bf16* vbase = p.v_cache + ((size_t)b * p.Hkv + hk) * p.P_cap * DH;

  // Q tile (rows >= R zero-filled)
  for (int i = tid; i < 64 * CH; i += 128) {
    const int row = i / CH, ch = i % CH;
    const bool ok = row < R;
    cp_async16(smem_u32(Qs + swz<DH>(row, ch)), ok ? (const void*)(qsrc + (size_t)row * DH + ch * 8) : (const void*)qsrc, ok ? 16 : 0);
  }
  auto load_tile = [&](int ti, int buf) {
    const int k0 = k_begin + ti * 64;
    for (int i = tid; i < 64 * CH; i += 128) {
      const int row = i / CH, ch = i % CH;
      const int kk = k0 + row;
      const bool ok = kk < k_end;
      const size_t off = (size_t)(ok ? kk : 0) * DH + ch * 8;
      cp_async16(smem_u32(Ks + buf * TILE_BYTES + swz<DH>(row, ch)), kbase + off, ok ? 16 : 0);
      cp_async16(smem_u32(Vs + buf * TILE_BYTES + swz<DH>(row, ch)), vbase + off, ok ? 16 : 0);
    }
  };
  load_tile(0, 0);
  cp_async_commit();

  const float sl2 = rsqrtf((float)DH) * 1.4426950408889634f;  // 1/sqrt(d_h) * log2(e)
  float o[DH / 8][4];
#pragma unroll
  for (int n = 0; n < DH / 8; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  uint32_t qf[DH / 16][4];
  const bool active = warp < n_mt;
  const int rr0 = warp * 16 + g, rr1 = rr0 + 8;
  const int lim0 = P + (rr0 % p.K), lim1 = P + (rr1 % p.K);  // last visible key position per row

  for (int ti = 0; ti < n_tiles; ++ti) {
    const int buf = ti & 1;
    if (ti + 1 < n_tiles) load_tile(ti + 1, buf ^ 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    if (active) {
      if (ti == 0) {
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks) {
          const int mi = lane >> 3;
          ldmatrix_x4(qf[ks], smem_u32(Qs + swz<DH>(warp * 16 + (mi & 1) * 8 + (lane & 7), 2 * ks + (mi >> 1))));
        }
      }
      float s[8][4];
#pragma unroll
      for (int n = 0; n < 8; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
      const unsigned char* Kt = Ks + buf * TILE_BYTES;
      const unsigned char* Vt = Vs + buf * TILE_BYTES;
#pragma unroll
      for (int ks = 0; ks < DH / 16; ++ks) {
#pragma unroll
        for (int np = 0; np < 4; ++np) {
          uint32_t kb[4];
          const int mi = lane >> 3;
          ldmatrix_x4(kb, smem_u32(Kt + swz<DH>(16 * np + (mi >> 1) * 8 + (lane & 7), 2 * ks + (mi & 1))));
          mma_bf16_16816(s[2 * np], qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], kb[0], kb[1]);
          mma_bf16_16816(s[2 * np + 1], qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], kb[2], kb[3]);
        }
      }
      // scale, mask, online softmax (rows g and g+8 of this warp's tile)
      const int k0 = k_begin + ti * 64;
      float tmax0 = -INFINITY, tmax1 = -INFINITY;
#pragma unroll
      for (int n = 0; n < 8; ++n) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int kk = k0 + n * 8 + 2 * t + e;
          const bool in = kk < k_end;
          s[n][e] = (in && kk <= lim0) ? s[n][e] * sl2 : -INFINITY;
          s[n][2 + e] = (in && kk <= lim1) ? s[n][2 + e] * sl2 : -INFINITY;
          tmax0 = fmaxf(tmax0, s[n][e]);
          tmax1 = fmaxf(tmax1, s[n][2 + e]);
        }
      }
      tmax0 = fmaxf(tmax0, __shfl_xor_sync(0xffffffffu, tmax0, 1));
      tmax0 = fmaxf(tmax0, __shfl_xor_sync(0xffffffffu, tmax0, 2));
      tmax1 = fmaxf(tmax1, __shfl_xor_sync(0xffffffffu, tmax1, 1));
      tmax1 = fmaxf(tmax1, __shfl_xor_sync(0xffffffffu, tmax1, 2));
      const float mn0 = fmaxf(m_run[0], tmax0), mn1 = fmaxf(m_run[1], tmax1);
      const float ms0 = (mn0 == -INFINITY) ? 0.f : mn0, ms1 = (mn1 == -INFINITY) ? 0.f : mn1;
      const float al0 = exp2f(m_run[0] - ms0), al1 = exp2f(m_run[1] - ms1);
      m_run[0] = mn0;
      m_run[1] = mn1;
      float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
      for (int n = 0; n < 8; ++n) {
        s[n][0] = exp2f(s[n][0] - ms0);
        s[n][1] = exp2f(s[n][1] - ms0);
        s[n][2] = exp2f(s[n][2] - ms1);
        s[n][3] = exp2f(s[n][3] - ms1);
        sum0 += s[n][0] + s[n][1];
        sum1 += s[n][2] + s[n][3];
      }
      l_run[0] = l_run[0] * al0 + sum0;
      l_run[1] = l_run[1] * al1 + sum1;
#pragma unroll
      for (int n = 0; n < DH / 8; ++n) {
        o[n][0] *= al0; o[n][1] *= al0; o[n][2] *= al1; o[n][3] *= al1;
      }
#pragma unroll
      for (int kp = 0; kp < 4; ++kp) {
        const uint32_t a0 = pack_bf16(s[2 * kp][0], s[2 * kp][1]), a1 = pack_bf16(s[2 * kp][2], s[2 * kp][3]);
        const uint32_t a2 = pack_bf16(s[2 * kp + 1][0], s[2 * kp + 1][1]), a3 = pack_bf16(s[2 * kp + 1][2], s[2 * kp + 1][3]);
#pragma unroll
        for (int dp = 0; dp < DH / 16; ++dp) {
          uint32_t vb[4];
          const int mi = lane >> 3;
          ldmatrix_x4_trans(vb, smem_u32(Vt + swz<DH>(16 * kp + (mi & 1) * 8 + (lane & 7), 2 * dp + (mi >> 1))));
          mma_bf16_16816(o[2 * dp], a0, a1, a2, a3, vb[0], vb[1]);
          mma_bf16_16816(o[2 * dp + 1], a0, a1, a2, a3, vb[2], vb[3]);
        }
      }
    }
    __syncthreads();
  }
  cp_async_wait<0>();
  if (!active) return;
  l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 1);
  l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 2);
  l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 1);
  l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 2);
  const size_t slot = ((size_t)(a.chunk_base[b] + ci) * p.Hkv + hk) * 64;
  float* op = p.o_part + slot * DH;
  float* mlp = p.ml_part + slot * 2;
  if (rr0 < R) {
#pragma unroll
    for (int n = 0; n < DH / 8; ++n)
      *reinterpret_cast<float2*>(op + (size_t)rr0 * DH + n * 8 + 2 * t) = make_float2(o[n][0], o[n][1]);
    if (t == 0) { mlp[rr0 * 2] = m_run[0]; mlp[rr0 * 2 + 1] = l_run[0]; }
  }
  if (rr1 < R) {
#pragma unroll
    for (int n = 0; n < DH / 8; ++n)
      *reinterpret_cast<float2*>(op + (size_t)rr1 * DH + n * 8 + 2 * t) = make_float2(o[n][2], o[n][3]);
    if (t == 0) { mlp[rr1 * 2] = m_run[1]; mlp[rr1 * 2 + 1] = l_run[1]; }
  }
}

// One block per (token row, query head): merge the chunk partials, normalise, emit hi/lo.
__global__ void attn_combine_kernel(const AttnArgs a) {
  const AttnParams& p = a.p;
  const int m = blockIdx.x, j = blockIdx.y, d = threadIdx.x, dh = p.dh;
  const int b = m / p.K, r = m % p.K, G = p.Hq / p.Hkv, hk = j / G, rr = (j % G) * p.K + r;
  const int n_chunks = a.chunk_base[b + 1] - a.chunk_base[b];
  float mx = -INFINITY;
  for (int c = 0; c < n_chunks; ++c) {
    const size_t slot = ((size_t)(a.chunk_base[b] + c) * p.Hkv + hk) * 64 + rr;
    mx = fmaxf(mx, p.ml_part[slot * 2]);
  }
  float L = 0.f, O = 0.f;
  for (int c = 0; c < n_chunks; ++c) {
    const size_t slot = ((size_t)(a.chunk_base[b] + c) * p.Hkv + hk) * 64 + rr;
    const float mc = p.ml_part[slot * 2];
    if (mc == -INFINITY) continue;
    const float wgt = exp2f(mc - mx);
    L += p.ml_part[slot * 2 + 1] * wgt;
    O += p.o_part[slot * dh + d] * wgt;
  }
  const float v = O / L;
  bf16 hi, lo;
  split_bf16(v, hi, lo);
  const size_t idx = (size_t)m * p.Hq * dh + (size_t)j * dh + d;
  p.a_hi[idx] = hi;
  p.a_lo[idx] = lo;
}

cudaError_t attention_setup() {
  return cudaFuncSetAttribute(attn_splitkv_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, 5 * 64 * 128 * 2);
}

cudaError_t launch_attention(const AttnParams& p, const int* seq_lens_host, cudaStream_t st) {
  AttnArgs a;
  a.p = p;
  int base = 0, max_chunks = 0;
  for (int b = 0; b < p.B; ++b) {
    a.chunk_base[b] = base;
    const int n = (seq_lens_host[b] + p.K + p.chunk_keys - 1) / p.chunk_keys;
    base += n;
    if (n > max_chunks) max_chunks = n;
  }
  a.chunk_base[p.B] = base;
  dim3 grid(max_chunks, p.Hkv, p.B);
  if (p.dh == 128)
    attn_splitkv_kernel<128><<<grid, 128, 5 * 64 * 128 * 2, st>>>(a);
  else
    attn_splitkv_kernel<64><<<grid, 128, 5 * 64 * 64 * 2, st>>>(a);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  dim3 cgrid(p.B * p.K, p.Hq);
  attn_combine_kernel<<<cgrid, p.dh, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace dart
