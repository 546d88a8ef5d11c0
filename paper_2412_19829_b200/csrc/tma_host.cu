// Host-side tensor-map construction for the TMA-fed kernels.
#include <mutex>

#include "common.cuh"
#include "sm100.cuh"

namespace gf {

EncodeTiledFn get_encode_tiled() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

bool make_qkv_tensor_map(CUtensorMap* map, const void* base, int B, int H, int N, int d, int layout,
                         int box_rows) {
  EncodeTiledFn enc = get_encode_tiled();
  if (!enc) return false;
  const Strides st = make_strides(layout, H, N, d);
  cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)N, (cuuint64_t)H, (cuuint64_t)B};
  cuuint64_t strides[3] = {(cuuint64_t)st.n * 2, (cuuint64_t)st.h * 2, (cuuint64_t)st.b * 2};
  cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Feature tensors are contiguous [B, h_count, N, d] and hold the heads [h_begin, h_begin + h_count) of
// the call.  The map addresses them with the call's own head coordinate h (as the Q, K, V, O maps
// do): the base is moved back by h_begin heads, which are never touched.
bool make_feature_tensor_map(CUtensorMap* map, const void* base, int B, int H, int N, int d, int h_begin,
                             int h_count, int box_rows) {
  EncodeTiledFn enc = get_encode_tiled();
  if (!enc) return false;
  const unsigned long long head_bytes = (unsigned long long)N * d * 2;
  const uintptr_t shifted = reinterpret_cast<uintptr_t>(base) - (uintptr_t)h_begin * head_bytes;
  cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)N, (cuuint64_t)H, (cuuint64_t)B};
  cuuint64_t strides[3] = {(cuuint64_t)d * 2, (cuuint64_t)head_bytes, (cuuint64_t)h_count * head_bytes};
  cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, reinterpret_cast<void*>(shifted), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace gf
