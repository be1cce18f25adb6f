// Host side of the tensor-core kernels: TMA tensor-map encoding through the driver entry point
// (looked up at run time so the library links against the CUDA runtime only).
#include <mutex>

#include "tc_common.cuh"

namespace isopo {
namespace tc {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  });
  return fn;
}

isopo_status make_map_2d_bf16(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols,
                              uint64_t row_stride_elems, uint32_t box_cols, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) {
    set_cuda_error(cudaErrorNotSupported, "cuTensorMapEncodeTiled entry point");
    return ISOPO_ERR_CUDA;
  }
  if (box_cols * 2 != 128 || box_rows == 0 || box_rows > 256 || (row_stride_elems * 2) % 16 != 0 ||
      ((uintptr_t)base & 15))
    return ISOPO_ERR_INVALID_ARG;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {row_stride_elems * 2};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return ISOPO_ERR_CUDA;
  }
  return ISOPO_OK;
}

isopo_status make_map_pieces_bf16(CUtensorMap* map, const void* base, uint64_t B, uint64_t pieces, uint32_t box_rows,
                                  uint32_t box_pieces) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) {
    set_cuda_error(cudaErrorNotSupported, "cuTensorMapEncodeTiled entry point");
    return ISOPO_ERR_CUDA;
  }
  if (box_rows == 0 || box_rows > 256 || box_pieces == 0 || box_pieces > 256 || ((uintptr_t)base & 15) || B == 0 ||
      pieces == 0)
    return ISOPO_ERR_INVALID_ARG;
  cuuint64_t dims[3] = {256, B, pieces};
  cuuint64_t strides[2] = {512, B * 512};
  cuuint32_t box[3] = {64, box_rows, box_pieces};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled (stored gradients)");
    return ISOPO_ERR_CUDA;
  }
  return ISOPO_OK;
}

isopo_status make_map_pieces_u8(CUtensorMap* map, const void* base, uint64_t B, uint64_t pieces, uint32_t box_rows,
                                uint32_t box_pieces) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) {
    set_cuda_error(cudaErrorNotSupported, "cuTensorMapEncodeTiled entry point");
    return ISOPO_ERR_CUDA;
  }
  if (box_rows == 0 || box_rows > 256 || box_pieces == 0 || box_pieces > 256 || ((uintptr_t)base & 15) || B == 0 ||
      pieces == 0)
    return ISOPO_ERR_INVALID_ARG;
  cuuint64_t dims[3] = {256, B, pieces};
  cuuint64_t strides[2] = {256, B * 256};
  cuuint32_t box[3] = {128, box_rows, box_pieces};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled (e4m3 plane)");
    return ISOPO_ERR_CUDA;
  }
  return ISOPO_OK;
}

}  // namespace tc
}  // namespace isopo
