// Split-KV grouped-query attention of the K query rows over the prefix KV cache and over each
// other (Section 3.1: strictly causal over the prefix and inside the masked block;
// Appendix B: grouped-query heads, post-RoPE keys in the cache).
//
// One CTA handles one (sequence, KV head, chunk of keys); its (H_q/H_kv)*K query rows (<= 64)
// form up to four 16-row MMA tiles, one per warp.  Cache chunks cover positions [0, P_b), which
// every query row may read; one extra chunk per sequence holds the step's own K new rows, read
// causally (row r reads new rows r' <= r).  KV tiles of 64 keys are staged in shared memory
// with cp.async (double buffered, XOR-swizzled 16-byte chunks); scores and P*V run on
// mma.sync.m16n8k16 with a warp-level online softmax; the per-chunk (max, sum, unnormalised
// output) partials are merged by attn_combine_kernel, which also emits the bf16 hi/lo
// activations for o_proj.
//
// Accuracy: the queries, the softmax weights and the new rows' k, v enter the bf16 MMAs as
// hi + lo pairs (x ~= hi + lo), so only the cache itself is bf16.  The new rows come from a
// 16-row side tile per (sequence, KV head): rows 0..7 hold the hi parts, rows 8..15 the lo
// parts, so the same MMA code produces q.k_hi in score columns 0..7 and q.k_lo in columns
// 8..15 (same thread, same register slot), which are added before the softmax; for P*V the
// weights of columns 0..7 are duplicated into 8..15 so that P*(v_hi + v_lo) falls out.
#include "common.cuh"
#include "kernels.h"

namespace dart {

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
// (a, b) -> packed bf16 hi parts and packed bf16 lo parts
__device__ __forceinline__ void pack_hi_lo(float a, float b, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  const __nv_bfloat162 l = __floats2bfloat162_rn(a - __low2float(h), b - __high2float(h));
  hi = *reinterpret_cast<const uint32_t*>(&h);
  lo = *reinterpret_cast<const uint32_t*>(&l);
}

// byte offset of 16-byte chunk `chunk` of row `row` in a [rows][DH] bf16 tile, XOR-swizzled
template <int DH>
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
  return (uint32_t)(row * (DH * 2) + ((chunk ^ (row & 7)) << 4));
}

template <int DH>
__global__ void __launch_bounds__(128) attn_splitkv_kernel(const __grid_constant__ AttnArgs a) {
  const AttnParams& p = a.p;
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int TILE_BYTES = 64 * DH * 2;
  constexpr int CH = DH / 8;  // 16-byte chunks per row
  unsigned char* Qh = smem;
  unsigned char* Ql = smem + TILE_BYTES;
  unsigned char* Ks = smem + 2 * TILE_BYTES;
  unsigned char* Vs = smem + 4 * TILE_BYTES;

  const int ci = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
  const int P = p.seq_lens[b];   // an input of the step: readable before the previous kernel has finished
  const int n_cc = (P + p.chunk_keys - 1) / p.chunk_keys;  // cache chunks of this sequence
  if (ci > n_cc) return;
  const bool is_new = ci == n_cc;
  const int k_begin = is_new ? 0 : ci * p.chunk_keys;
  const int k_end = is_new ? 16 : min(P, k_begin + p.chunk_keys);
  const int n_tiles = (k_end - k_begin + 63) >> 6;
  const int G = p.Hq / p.Hkv, R = G * p.K;
  const int n_mt = (R + 15) >> 4;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;

  const size_t qoff = ((size_t)b * p.Hq + (size_t)hk * G) * p.K * DH;
  const bf16* kbase = is_new ? p.k_new + ((size_t)b * p.Hkv + hk) * 16 * DH
                             : p.k_cache + ((size_t)b * p.Hkv + hk) * p.P_cap * DH;
  const bf16* vbase = is_new ? p.v_new + ((size_t)b * p.Hkv + hk) * 16 * DH
                             : p.v_cache + ((size_t)b * p.Hkv + hk) * p.P_cap * DH;

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
  // Cache rows below P_b were written by earlier steps, so a cache chunk's first tile is requested while the
  // QKV kernel is still finishing; q and the new rows' side tile are its outputs and wait for it.
  if (!is_new) load_tile(0, 0);
  cp_async_commit();
  pdl_wait();
  pdl_trigger();   // a short kernel: the next one may be scheduled and run its set-up now
  // Q tiles, hi and lo (rows >= R zero-filled)
  for (int i = tid; i < 64 * CH; i += 128) {
    const int row = i / CH, ch = i % CH;
    const bool ok = row < R;
    const size_t off = qoff + (ok ? (size_t)row * DH + ch * 8 : 0);
    cp_async16(smem_u32(Qh + swz<DH>(row, ch)), p.q_hi + off, ok ? 16 : 0);
    cp_async16(smem_u32(Ql + swz<DH>(row, ch)), p.q_lo + off, ok ? 16 : 0);
  }
  if (is_new) load_tile(0, 0);
  cp_async_commit();

  const float sl2 = rsqrtf((float)DH) * 1.4426950408889634f;  // 1/sqrt(d_h) * log2(e)
  float o[DH / 8][4];
#pragma unroll
  for (int n = 0; n < DH / 8; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  const bool active = warp < n_mt;
  const int rr0 = warp * 16 + g, rr1 = rr0 + 8;
  const int r0 = rr0 % p.K, r1 = rr1 % p.K;  // position of the row inside its sequence's K-block

  for (int ti = 0; ti < n_tiles; ++ti) {
    const int buf = ti & 1;
    if (ti + 1 < n_tiles) load_tile(ti + 1, buf ^ 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    if (active) {
      float s[8][4];
#pragma unroll
      for (int n = 0; n < 8; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
      const unsigned char* Kt = Ks + buf * TILE_BYTES;
      const unsigned char* Vt = Vs + buf * TILE_BYTES;
      const int mi = lane >> 3;
#pragma unroll
      for (int ks = 0; ks < DH / 16; ++ks) {
        uint32_t qh[4], ql[4];
        const uint32_t qa = swz<DH>(warp * 16 + (mi & 1) * 8 + (lane & 7), 2 * ks + (mi >> 1));
        ldmatrix_x4(qh, smem_u32(Qh + qa));
        ldmatrix_x4(ql, smem_u32(Ql + qa));
#pragma unroll
        for (int np = 0; np < 4; ++np) {
          if (is_new && np > 0) break;  // the new-rows tile has 16 rows only
          uint32_t kb[4];
          ldmatrix_x4(kb, smem_u32(Kt + swz<DH>(16 * np + (mi >> 1) * 8 + (lane & 7), 2 * ks + (mi & 1))));
          mma_bf16_16816(s[2 * np], qh[0], qh[1], qh[2], qh[3], kb[0], kb[1]);
          mma_bf16_16816(s[2 * np], ql[0], ql[1], ql[2], ql[3], kb[0], kb[1]);
          mma_bf16_16816(s[2 * np + 1], qh[0], qh[1], qh[2], qh[3], kb[2], kb[3]);
          mma_bf16_16816(s[2 * np + 1], ql[0], ql[1], ql[2], ql[3], kb[2], kb[3]);
        }
      }
      // scale, mask, online softmax (rows g and g+8 of this warp's tile)
      const int k0 = k_begin + ti * 64;
      float tmax0 = -INFINITY, tmax1 = -INFINITY;
      if (is_new) {
#pragma unroll
        for (int e = 0; e < 4; ++e) s[0][e] += s[1][e];  // q.k_hi + q.k_lo
      }
#pragma unroll
      for (int n = 0; n < 8; ++n) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int kk = k0 + n * 8 + 2 * t + e;
          // cache chunk: every position below P is visible; new chunk: column r' (< K) visible to rows r >= r'
          const bool v0 = is_new ? (n == 0 && kk < p.K && kk <= r0) : (kk < k_end);
          const bool v1 = is_new ? (n == 0 && kk < p.K && kk <= r1) : (kk < k_end);
          s[n][e] = v0 ? s[n][e] * sl2 : -INFINITY;
          s[n][2 + e] = v1 ? s[n][2 + e] * sl2 : -INFINITY;
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
      if (is_new) {
#pragma unroll
        for (int e = 0; e < 4; ++e) s[1][e] = s[0][e];  // same weights on the v_lo rows
      }
#pragma unroll
      for (int n = 0; n < DH / 8; ++n) {
        o[n][0] *= al0; o[n][1] *= al0; o[n][2] *= al1; o[n][3] *= al1;
      }
#pragma unroll
      for (int kp = 0; kp < 4; ++kp) {
        if (is_new && kp > 0) break;
        uint32_t ah[4], al[4];
        pack_hi_lo(s[2 * kp][0], s[2 * kp][1], ah[0], al[0]);
        pack_hi_lo(s[2 * kp][2], s[2 * kp][3], ah[1], al[1]);
        pack_hi_lo(s[2 * kp + 1][0], s[2 * kp + 1][1], ah[2], al[2]);
        pack_hi_lo(s[2 * kp + 1][2], s[2 * kp + 1][3], ah[3], al[3]);
#pragma unroll
        for (int dp = 0; dp < DH / 16; ++dp) {
          uint32_t vb[4];
          ldmatrix_x4_trans(vb, smem_u32(Vt + swz<DH>(16 * kp + (mi & 1) * 8 + (lane & 7), 2 * dp + (mi >> 1))));
          mma_bf16_16816(o[2 * dp], ah[0], ah[1], ah[2], ah[3], vb[0], vb[1]);
          mma_bf16_16816(o[2 * dp], al[0], al[1], al[2], al[3], vb[0], vb[1]);
          mma_bf16_16816(o[2 * dp + 1], ah[0], ah[1], ah[2], ah[3], vb[2], vb[3]);
          mma_bf16_16816(o[2 * dp + 1], al[0], al[1], al[2], al[3], vb[2], vb[3]);
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

// One block per (token row, query head): merge the chunk partials, normalise, emit hi/lo.  The block is
// four groups of d_h threads; the (max, sum) pairs of all chunks are fetched in one round of loads, the
// groups then add up interleaved quarters of the chunks' outputs (independent loads, one more round) and
// their four partial sums are added in a fixed order.
constexpr int kMaxChunks = 192;   // chunks per sequence the combine can hold (host checks)

__global__ void attn_combine_kernel(const AttnArgs a) {
  const AttnParams& p = a.p;
  __shared__ float s_m[kMaxChunks], s_w[kMaxChunks];
  __shared__ float s_o[4][128];
  __shared__ float s_L;
  const int m = blockIdx.x, j = blockIdx.y, dh = p.dh, tid = threadIdx.x, g = tid / dh, d = tid - g * dh;
  const int b = m / p.K, r = m % p.K, G = p.Hq / p.Hkv, hk = j / G, rr = (j % G) * p.K + r;
  const int n_chunks = a.chunk_base[b + 1] - a.chunk_base[b];
  const size_t slot0 = ((size_t)a.chunk_base[b] * p.Hkv + hk) * 64 + rr, slot_step = (size_t)p.Hkv * 64;
  pdl_wait();
  pdl_trigger();   // a short kernel: the next one may be scheduled and run its set-up now
  float l_c = 0.f;
  if (tid < n_chunks) {
    const float2 ml = *reinterpret_cast<const float2*>(p.ml_part + (slot0 + (size_t)tid * slot_step) * 2);
    s_m[tid] = ml.x;
    l_c = ml.y;
  }
  __syncthreads();
  float mx = -INFINITY;
  for (int c = 0; c < n_chunks; ++c) mx = fmaxf(mx, s_m[c]);
  if (tid < n_chunks) s_w[tid] = s_m[tid] == -INFINITY ? 0.f : exp2f(s_m[tid] - mx);
  __syncthreads();
  // L = sum of l_c * w_c in chunk order: the products go through s_m (its maxima are no longer needed)
  if (tid < n_chunks) s_m[tid] = l_c * s_w[tid];
  __syncthreads();
  if (tid == 0) {
    float L = 0.f;
    for (int c = 0; c < n_chunks; ++c) L += s_m[c];
    s_L = L;
  }
  float O = 0.f;
  const float* op = p.o_part + slot0 * dh + d;
#pragma unroll 4
  const int n_groups = blockDim.x / dh;
  for (int c = g; c < n_chunks; c += n_groups) {
    const float w = s_w[c];
    if (w != 0.f) O += op[(size_t)c * slot_step * dh] * w;
  }
  s_o[g][d] = O;
  if (g == 0)
    for (int q = n_groups; q < 4; ++q) s_o[q][d] = 0.f;
  __syncthreads();
  if (g == 0) {
    const float v = (((s_o[0][d] + s_o[1][d]) + s_o[2][d]) + s_o[3][d]) / s_L;
    bf16 hi, lo;
    split_bf16(v, hi, lo);
    const size_t idx = (size_t)m * p.Hq * dh + (size_t)j * dh + d;
    p.a_hi[idx] = hi;
    p.a_lo[idx] = lo;
  }
}

cudaError_t attention_setup() {
  cudaError_t e = cudaFuncSetAttribute(attn_splitkv_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, 6 * 64 * 128 * 2);
  return e != cudaSuccess ? e : attn_umma_setup();
}

// Whether the step's attention runs on the tcgen05 split (attn_umma.cu).  It pays a few microseconds of set-up per
// CTA (barriers, tensor memory, first loads) and wins from about 512 (64-key tile, KV head) pairs on (attention stage,
// split and combine: batch 1 x 4096 keys x 8 heads 21.5 vs 23.6 us; 2048 keys 21.7 vs 21.5; batch 4 x 8192 keys 49.6
// vs 89).
bool attn_uses_umma(int B, int Hkv, int dh, const int* seq_lens_host, bool have_maps) {
  long long key_tiles = 0;
  for (int b = 0; b < B; ++b) key_tiles += (seq_lens_host[b] + 63) / 64;
  return have_maps && dh == 128 && key_tiles * Hkv >= 512;
}

// Chunk length for the tcgen05 split, whose CTAs take two consecutive chunks of a sequence each and stay alone on
// their SM.  Short chunks mean several waves of CTAs, each paying its set-up, and more partials for the combine; long
// ones leave SMs idle or one CTA with a long tail.  The estimate below -- a CTA costs its first chunk's 64-key tiles
// plus six tiles' worth of set-up; one wave lasts as long as its longest CTA, more waves as long as the work spread
// over the SMs plus half a CTA -- reproduces the measured order (4 x 8192 keys, 8 KV heads: 1216 keys 48 us, 1024:
// 52, 512: 58; 16 ragged sequences: 1408 keys 103 us, 1024: 107, 512: 120, 4096: 146).  Candidates are the multiples
// of 64 from 128 to 2048 whose chunk count fits `pairs_cap`; returns 0 if none does.
int attn_umma_chunk_keys(int B, int Hkv, const int* seq_lens_host, int n_sm, int pairs_cap) {
  constexpr int kSetupTiles = 6;
  int best = 0;
  double best_t = 0.0;
  for (int chunk = 128; chunk <= 2048; chunk += 64) {
    long long ctas = 0, total = 0, pairs = 0;
    int longest = 0, most = 0;
    for (int b = 0; b < B; ++b) {
      const int P = seq_lens_host[b];
      const int ncc = (P + chunk - 1) / chunk;            // cache chunks; chunk ncc is the new rows
      const int n_full = ncc > 0 ? ncc / 2 : 0;           // CTAs whose first chunk is a whole one: 2x < ncc - 1
      const int full_cost = chunk / 64 + kSetupTiles;
      // the last CTA starts with the sequence's last cache chunk (ncc odd) or with the new rows (ncc even)
      const int last_tiles = (ncc & 1) ? (P - (ncc - 1) * chunk + 63) / 64 : 1;
      const int last_cost = last_tiles + kSetupTiles;
      ctas += n_full + 1;
      total += (long long)n_full * full_cost + last_cost;
      if (n_full > 0 && full_cost > longest) longest = full_cost;
      if (last_cost > longest) longest = last_cost;
      pairs += ncc + 1;
      if (ncc + 1 > most) most = ncc + 1;
    }
    if (pairs > pairs_cap || most > kMaxChunks) continue;
    ctas *= Hkv; total *= Hkv;
    const double spread = (double)total / n_sm + 0.5 * longest;
    const double t = ctas <= n_sm ? (double)longest : (spread > longest ? spread : (double)longest);
    if (best == 0 || t < best_t) { best = chunk; best_t = t; }
  }
  return best;
}

cudaError_t launch_attention(const AttnParams& p, const int* seq_lens_host, const AttnUmmaMaps* maps, int* status, cudaStream_t st) {
  AttnArgs a;
  a.p = p;
  int base = 0, max_chunks = 0;
  for (int b = 0; b < p.B; ++b) {
    a.chunk_base[b] = base;
    const int n = (seq_lens_host[b] + p.chunk_keys - 1) / p.chunk_keys + 1;  // cache chunks + the new-rows chunk
    base += n;
    if (n > max_chunks) max_chunks = n;
  }
  a.chunk_base[p.B] = base;
  if (max_chunks > kMaxChunks) return cudaErrorInvalidValue;
  dim3 grid(max_chunks, p.Hkv, p.B);
  cudaError_t e;
  if (attn_uses_umma(p.B, p.Hkv, p.dh, seq_lens_host, maps != nullptr)) {
    AttnUmmaArgs u;
    u.a = a;
    u.mapQhi = maps->mapQhi; u.mapQlo = maps->mapQlo; u.mapK = maps->mapK; u.mapV = maps->mapV; u.mapKn = maps->mapKn; u.mapVn = maps->mapVn;
    u.status = status;
    e = launch_attn_umma_split(u, max_chunks, st);
  } else if (p.dh == 128)
    e = launch_pdl(attn_splitkv_kernel<128>, grid, dim3(128), (size_t)6 * 64 * 128 * 2, st, a);
  else
    e = launch_pdl(attn_splitkv_kernel<64>, grid, dim3(128), (size_t)6 * 64 * 64 * 2, st, a);
  if (e != cudaSuccess) return e;
  dim3 cgrid(p.B * p.K, p.Hq);
  // few chunks per sequence: one thread per output column walks all of them (one barrier less, more blocks per SM);
  // many chunks: four groups of d_h threads share them (measured: 17 chunks 159 vs 175 us, 33 chunks 29.5 vs 23.6 us)
  const int groups = max_chunks <= 20 ? 1 : 4;
  return launch_pdl(attn_combine_kernel, cgrid, dim3(groups * p.dh), 0, st, a);
}

}  // namespace dart
