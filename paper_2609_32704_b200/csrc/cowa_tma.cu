#include "cowa_tma.h"

namespace cowa {

namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  // The driver entry point is resolved at run time so that the library links without libcuda.
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}
}  // namespace

int make_tensor_map(CUtensorMap* map, const void* base, MapType type, int D, long long T, int H, int B,
                    const CowaStrides& st, int box_d, int box_t, bool swizzle128) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return record_cuda_error(cudaErrorNotSupported);
  const size_t es = type == MapType::BF16 ? 2 : 4;
  cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)T, (cuuint64_t)H, (cuuint64_t)B};
  // a dimension of extent 1 is never stepped along: give it a harmless stride when the caller left it at 0
  const cuuint64_t row = (cuuint64_t)D * es;
  cuuint64_t strides[3] = {(cuuint64_t)st.t * es, (cuuint64_t)st.h * es, (cuuint64_t)st.b * es};
  for (cuuint64_t& x : strides)
    if (x == 0) x = row;
  cuuint32_t box[4] = {(cuuint32_t)box_d, (cuuint32_t)box_t, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  const CUtensorMapDataType dt = type == MapType::BF16  ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                                 : type == MapType::F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                                        : CU_TENSOR_MAP_DATA_TYPE_INT32;
  CUresult r = fn(map, dt, 4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return record_cuda_error(cudaErrorInvalidValue);
  return COWA_OK;
}

}  // namespace cowa
