// Host-side tensor-map construction for the TMA-fed kernels.
#include <string.h>

#include <mutex>
#include <vector>

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

cudaError_t device_info(int* dev, int* sms) {
  constexpr int kMaxDev = 64;
  static int cached[kMaxDev];  // 0 = not asked yet (a benign race: every writer stores the same value)
  cudaError_t e = cudaGetDevice(dev);
  if (e != cudaSuccess) return e;
  if (*dev < 0 || *dev >= kMaxDev) return cudaErrorInvalidDevice;
  int n = cached[*dev];
  if (n == 0) {
    if ((e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, *dev)) != cudaSuccess) return e;
    cached[*dev] = n;
  }
  *sms = n;
  return cudaSuccess;
}

cudaError_t ensure_dynamic_smem(const void* kernel, int dev, int bytes) {
  struct Done {
    const void* kernel;
    int dev, bytes;
  };
  static std::mutex mu;
  static std::vector<Done> done;
  {
    std::lock_guard<std::mutex> lock(mu);
    for (const Done& x : done)
      if (x.kernel == kernel && x.dev == dev && x.bytes >= bytes) return cudaSuccess;
  }
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return e;
  std::lock_guard<std::mutex> lock(mu);
  done.push_back(Done{kernel, dev, bytes});
  return cudaSuccess;
}

namespace {
// A tensor map depends on the address and the geometry only, so the last few are kept per host thread:
// a layer called again on the same buffers (the usual case) encodes nothing.
struct MapKey {
  const void* base;
  int B, H, N, d, a, b, box_rows, kind;
};
struct MapCache {
  static constexpr int kEntries = 16;
  MapKey key[kEntries];
  CUtensorMap map[kEntries];
  int used = 0, next = 0;
  const CUtensorMap* find(const MapKey& k) const {
    for (int i = 0; i < used; ++i)
      if (memcmp(&key[i], &k, sizeof(MapKey)) == 0) return &map[i];
    return nullptr;
  }
  void put(const MapKey& k, const CUtensorMap& m) {
    const int i = used < kEntries ? used++ : (next++ % kEntries);
    key[i] = k;
    map[i] = m;
  }
};
thread_local MapCache t_maps;
MapKey map_key(const void* base, int B, int H, int N, int d, int a, int b, int box_rows, int kind) {
  MapKey k;
  memset(&k, 0, sizeof(k));  // padding bytes take part in the comparison
  k.base = base;
  k.B = B;
  k.H = H;
  k.N = N;
  k.d = d;
  k.a = a;
  k.b = b;
  k.box_rows = box_rows;
  k.kind = kind;
  return k;
}
}  // namespace

bool make_qkv_tensor_map(CUtensorMap* map, const void* base, int B, int H, int N, int d, int layout,
                         int box_rows) {
  const MapKey key = map_key(base, B, H, N, d, layout, 0, box_rows, 0);
  if (const CUtensorMap* hit = t_maps.find(key)) {
    *map = *hit;
    return true;
  }
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
  if (r == CUDA_SUCCESS) t_maps.put(key, *map);
  return r == CUDA_SUCCESS;
}

// Feature tensors are contiguous [B, h_count, N, d] and hold the heads [h_begin, h_begin + h_count) of
// the call.  The map addresses them with the call's own head coordinate h (as the Q, K, V, O maps
// do): the base is moved back by h_begin heads, which are never touched.
bool make_feature_tensor_map(CUtensorMap* map, const void* base, int B, int H, int N, int d, int h_begin,
                             int h_count, int box_rows) {
  const MapKey key = map_key(base, B, H, N, d, h_begin, h_count, box_rows, 1);
  if (const CUtensorMap* hit = t_maps.find(key)) {
    *map = *hit;
    return true;
  }
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
  if (r == CUDA_SUCCESS) t_maps.put(key, *map);
  return r == CUDA_SUCCESS;
}

}  // namespace gf
