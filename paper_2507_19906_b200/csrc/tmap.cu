// Host-side construction of TMA tensor maps.  The driver entry point is resolved through the
// runtime, so the library does not link against libcuda.
#include <cudaTypedefs.h>
#include <mutex>

#include "tc_common.cuh"

namespace calidrop {

namespace {

PFN_cuTensorMapEncodeTiled_v12000 resolve_encode() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
  });
  return fn;
}

}  // namespace

bool make_tensor_map_bf16(CUtensorMap* out, const void* base, int rank, const uint64_t* dims_from_1,
                          const uint64_t* strides_from_1, const uint32_t* box_from_1) {
  auto encode = resolve_encode();
  if (!encode || rank < 2 || rank > 5) return false;
  cuuint64_t dims[5] = {(cuuint64_t)kD, 1, 1, 1, 1};
  cuuint64_t strides[4] = {0, 0, 0, 0};
  cuuint32_t box[5] = {(cuuint32_t)tc::kHalfCols, 1, 1, 1, 1};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  for (int i = 1; i < rank; ++i) {
    dims[i] = dims_from_1[i - 1];
    strides[i - 1] = strides_from_1[i - 1];
    box[i] = box_from_1[i - 1];
    if (box[i] < 1 || box[i] > 256 || dims[i] < 1 || (strides[i - 1] & 15u)) return false;
  }
  const CUresult r = encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), dims,
                            strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace calidrop
