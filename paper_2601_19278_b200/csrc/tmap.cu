// Tensor maps for the TMA loads of the streaming kernels.  The encoder is a driver-API function; it is
// looked up through the runtime (cudaGetDriverEntryPoint), so the library needs no link against libcuda.
#include "kernels.h"

namespace dart {

namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encoder() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
      return nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}
}  // namespace

cudaError_t tmap_encode_bf16(CUtensorMap* m, const void* base, unsigned long long inner, unsigned long long outer,
                             unsigned long long ld_bytes, unsigned box_inner, unsigned box_outer) {
  EncodeTiledFn enc = encoder();
  if (enc == nullptr) return cudaErrorNotSupported;
  // the copy engine's rules: 16-byte aligned base and row stride, inner box extent of at most 128 bytes
  // for the 128-byte swizzle, box extents of at most 256 elements
  if ((reinterpret_cast<uintptr_t>(base) & 15u) != 0 || (ld_bytes & 15u) != 0 || box_inner * 2 > 128 || box_outer > 256 || inner == 0 ||
      outer == 0)
    return cudaErrorInvalidValue;
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {ld_bytes};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t elem[2] = {1, 1};
  const CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// hi and lo parts of an activation matrix as ONE 3-D tensor [rows][2][inner]: the lo buffer lies `pair_bytes` after
// the hi buffer, rows are ld_bytes apart.  A box {64, 2, box_rows} lands in shared memory as rows (hi, lo) of token
// 0, (hi, lo) of token 1, ...: one copy instead of two per stage.
cudaError_t tmap_encode_bf16_pair(CUtensorMap* m, const void* hi, unsigned long long pair_bytes, unsigned long long inner,
                                  unsigned long long rows, unsigned long long ld_bytes, unsigned box_rows) {
  EncodeTiledFn enc = encoder();
  if (enc == nullptr) return cudaErrorNotSupported;
  if ((reinterpret_cast<uintptr_t>(hi) & 15u) != 0 || (ld_bytes & 15u) != 0 || (pair_bytes & 15u) != 0 || pair_bytes == 0 || box_rows > 256 ||
      inner == 0 || rows == 0)
    return cudaErrorInvalidValue;
  cuuint64_t dims[3] = {inner, 2, rows};
  cuuint64_t strides[2] = {pair_bytes, ld_bytes};
  cuuint32_t box[3] = {64, 2, box_rows};
  cuuint32_t elem[3] = {1, 1, 1};
  const CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(hi), dims, strides, box, elem,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

}  // namespace dart
