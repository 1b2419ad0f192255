// Tensor-map (TMA descriptor) encoding on the host.  The driver entry point is resolved
// at run time so the library carries no link-time dependency on libcuda.
#include <cudaTypedefs.h>

#include "runtime.h"

namespace lv {

bool resolve_encode_tiled(void** fn) {
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
  if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || p == nullptr) {
    (void)cudaGetLastError();
    return false;
  }
  *fn = p;
  return true;
}

static bool encode_bf16_2d(void* encode_fn, CUtensorMap* out, const void* base, uint64_t inner, uint64_t outer,
                           uint64_t pitch_elems, uint32_t box_inner, uint32_t box_outer, CUtensorMapSwizzle swizzle) {
  auto encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(encode_fn);
  const cuuint64_t dims[2] = {inner, outer};
  const cuuint64_t strides[1] = {pitch_elems * 2};  // bytes, dimension 1
  const cuuint32_t box[2] = {box_inner, box_outer};
  const cuuint32_t elem_strides[2] = {1, 1};
  CUresult r = encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                      elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool make_tmap_bf16_2d(void* encode_fn, CUtensorMap* out, const void* base, uint64_t inner, uint64_t outer,
                       uint64_t pitch_elems, uint32_t box_inner, uint32_t box_outer) {
  return encode_bf16_2d(encode_fn, out, base, inner, outer, pitch_elems, box_inner, box_outer,
                        CU_TENSOR_MAP_SWIZZLE_128B);
}

// 2-D tensor of bytes [outer, inner] with row pitch `pitch_bytes`; box [box_outer, box_inner bytes];
// 64-byte swizzle for boxes whose rows are 64 bytes, 128-byte swizzle otherwise; zero fill outside.
bool make_tmap_u8_2d(void* encode_fn, CUtensorMap* out, const void* base, uint64_t inner, uint64_t outer,
                     uint64_t pitch_bytes, uint32_t box_inner, uint32_t box_outer) {
  auto encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(encode_fn);
  const cuuint64_t dims[2] = {inner, outer};
  const cuuint64_t strides[1] = {pitch_bytes};
  const cuuint32_t box[2] = {box_inner, box_outer};
  const cuuint32_t elem_strides[2] = {1, 1};
  const CUtensorMapSwizzle swizzle = box_inner == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B;
  CUresult r = encode(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, elem_strides,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace lv
