// Entry point for callers that cannot allocate device memory.
//
// Some hosts hand this library a stream and tensors but may not call cudaMalloc themselves: code
// running inside a memory pool that owns the whole device, a plug-in that must not touch the
// allocator of the framework it lives in, or a real-time loop where an allocation (and the
// implicit synchronisation it brings) is not acceptable.  The tensor-core linear-attention kernel
// needs scratch for the states its CTAs hand from segment to segment; here that scratch is a
// fixed array inside the library image instead of a caller-provided workspace.
#include <mutex>

#include "common.cuh"

namespace {

constexpr size_t kScratchBytes = 8u << 20;  // 8 MiB, resident on every GPU that loads the library
constexpr int kMaxDevices = 64;

// In host code this name is only a handle for the symbol; the device address is obtained with
// cudaGetSymbolAddress, once per device, with that device current.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

void* g_scratch_ptr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

// Returns the device address of the scratch array on the current device (nullptr on failure).
void* scratch_for_current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (g_scratch_ptr[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess) return nullptr;
    g_scratch_ptr[dev] = ptr;
  }
  return g_scratch_ptr[dev];
}

}  // namespace

extern "C" {

size_t gformer_noalloc_scratch_bytes(void) { return kScratchBytes; }

int gformer_causal_linear_attn_noalloc(const void* q, const void* k, const void* v, void* o, int B, int H, int N,
                                       int d, int phi, int chunk, float* S_io, float* z_io, int dtype, int layout,
                                       void* cuda_stream) {
  if (B < 1 || H < 1 || N < 1) return GF_ERR_INVALID_ARG;
  // Reject what does not fit before anything is touched: the array cannot grow.
  const size_t need = gformer_workspace_bytes(B, H, N, d, 1, 0, dtype);
  if (need > kScratchBytes) return GF_ERR_WORKSPACE;
  void* ws = scratch_for_current_device();
  if (ws == nullptr) return GF_ERR_CUDA;
  return gformer_causal_linear_attn(q, k, v, o, B, H, N, d, phi, chunk, S_io, z_io, dtype, layout, ws, kScratchBytes,
                                    cuda_stream);
}

// The status word of the fixed scratch (the workspace is hidden from the caller, so
// gformer_last_device_status cannot be pointed at it).
int gformer_noalloc_last_device_status(void* cuda_stream) {
  void* ws = scratch_for_current_device();
  if (ws == nullptr) return GF_ERR_CUDA;
  return gformer_last_device_status(ws, cuda_stream);
}

}  // extern "C"
