// Host-side construction of bf16 TMA tensor maps (128-byte swizzle).
// The driver entry point is fetched at run time so the library has no link-time
// dependency on libcuda.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>

namespace cpmtp {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode_fn() {
  // looked up once; initialisation of a function-local static is thread-safe
  static const EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess) {
      return reinterpret_cast<EncodeTiledFn>(p);
    }
    return nullptr;
  }();
  return fn;
}

// A row-major bf16 matrix [outer, inner] with `row_stride` elements between rows,
// read in boxes of box_inner x box_outer elements (box_inner * 2 bytes must be 128).
// Out-of-range elements read as zero.  Returns false on failure.
inline bool make_tmap_bf16(CUtensorMap* out, const void* base, uint64_t inner, uint64_t outer,
                           uint64_t row_stride, uint32_t box_inner, uint32_t box_outer) {
  EncodeTiledFn fn = get_encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {row_stride * 2};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t elem[2] = {1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// K-major A operand whose rows come in groups of `r` that are padded to `R` >= r tile rows:
// matrix [groups * r, k] viewed as [groups][r][k]; a box holds 64 (k) x R x groups_per_box and the
// rows r..R-1 of every group, like everything else out of range, read as zero.  The box lands in
// shared memory as groups_per_box * R dense 128-byte rows, i.e. as an ordinary row tile.
inline bool make_grouped_tmap_bf16(CUtensorMap* out, const void* base, uint64_t k, uint64_t r, uint64_t groups,
                                   uint64_t ld, uint32_t R, uint32_t groups_per_box) {
  EncodeTiledFn fn = get_encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[3] = {k, r, groups};
  cuuint64_t strides[2] = {ld * 2, ld * 2 * r};
  cuuint32_t box[3] = {64, R, groups_per_box};
  cuuint32_t elem[3] = {1, 1, 1};
  CUresult rc = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, elem,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS;
}

// Operand of D = A * B^T as the GEMM engine reads it.
//   K-major : matrix [rows, K] with K contiguous; tile box = 64 (K) x tile_rows
//   MN-major: matrix [K, rows] with the row index contiguous; tile box = 64 (rows) x 64 (K)
inline bool make_operand_tmap(CUtensorMap* out, const void* base, bool mn_major, uint64_t rows, uint64_t k,
                              uint64_t ld, uint32_t tile_rows) {
  if (!mn_major) return make_tmap_bf16(out, base, k, rows, ld, 64, tile_rows);
  return make_tmap_bf16(out, base, rows, k, ld, 64, 64);
}

}  // namespace cpmtp
