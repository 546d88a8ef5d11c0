// C ABI of libgformer: argument validation, path selection and launches.
#include <math.h>
#include <stdint.h>

#include <atomic>
#include <mutex>

#include "common.cuh"

namespace gf {
static std::atomic<unsigned long long> g_launches{0};
void note_launch(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }
}  // namespace gf

namespace {

using gf::Strides;
using gf::WsHeader;

// Process-wide knobs (gformer_set_tuning).  An entry point takes one snapshot when it is called
// and works from that, so a knob changed by another thread meanwhile cannot make the parts of one
// call disagree (the cleared flag bytes, the plan, the launch).
std::atomic<int> g_force_simt{0}, g_linear_split{0}, g_linear_ctas{0}, g_wait_kcycles{0}, g_drop_flag{0};
struct Tuning {
  int force_simt, linear_split, linear_ctas, wait_kcycles, drop_flag;
};
Tuning tuning_now() {
  Tuning t;
  t.force_simt = g_force_simt.load(std::memory_order_relaxed);
  t.linear_split = g_linear_split.load(std::memory_order_relaxed);
  t.linear_ctas = g_linear_ctas.load(std::memory_order_relaxed);
  t.wait_kcycles = g_wait_kcycles.load(std::memory_order_relaxed);
  t.drop_flag = g_drop_flag.load(std::memory_order_relaxed);
  return t;
}

constexpr int kMaxDevices = 64;
constexpr unsigned int kPlacedWaitNs = 20000;  // longest the windowed heads are held back for the linear kernel's CTAs
struct Fork {
  cudaStream_t side = nullptr, first = nullptr;  // lowest / highest stream priority
  cudaEvent_t fork = nullptr, join = nullptr, join_first = nullptr;
  bool ready = false;
  // held while a call enqueues its fork .. join section: the events are shared by every call on
  // the device, and a record from another host thread between this call's record and its waits
  // would make the side streams wait for the wrong point
  std::mutex enqueue;
};
Fork g_fork[kMaxDevices];
std::mutex g_fork_mutex;

// Side stream + two events per device, created on first use; lets the two head groups of the
// hybrid layer run concurrently while the caller sees a single-stream call.
Fork* get_fork() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_fork_mutex);
  Fork& f = g_fork[dev];
  if (!f.ready) {
    // lowest priority: where the two kernels compete for an SM, the persistent linear kernel
    // (whose CTAs wait for one another) is placed first
    int prio_least = 0, prio_greatest = 0;
    if (cudaDeviceGetStreamPriorityRange(&prio_least, &prio_greatest) != cudaSuccess) return nullptr;
    if (cudaStreamCreateWithPriority(&f.side, cudaStreamNonBlocking, prio_least) != cudaSuccess) return nullptr;
    if (cudaStreamCreateWithPriority(&f.first, cudaStreamNonBlocking, prio_greatest) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&f.join_first, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&f.fork, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&f.join, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    f.ready = true;
  }
  return &f;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool overlaps(const void* a, const void* b, size_t bytes) {
  const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
  return x < y + bytes && y < x + bytes;
}

size_t elem_size(int dtype) { return dtype == GF_F32 ? 4 : 2; }

int check_common(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d, int dtype,
                 int layout) {
  if (!q || !k || !v || !o) return GF_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return GF_ERR_INVALID_ARG;
  if (B < 1 || H < 1 || N < 1 || d < 1) return GF_ERR_INVALID_ARG;
  if (dtype != GF_F32 && dtype != GF_BF16) return GF_ERR_INVALID_ARG;
  if (layout != GF_BHND && layout != GF_BNHD) return GF_ERR_INVALID_ARG;
  if (d != 64 && d != 128) return GF_ERR_UNSUPPORTED;
  if ((long long)B * H > 65535LL * 65535LL || B > 65535 || H > 65535) return GF_ERR_UNSUPPORTED;
  const size_t bytes = (size_t)B * H * N * d * elem_size(dtype);
  if (overlaps(o, q, bytes) || overlaps(o, k, bytes) || overlaps(o, v, bytes)) return GF_ERR_INVALID_ARG;
  return GF_OK;
}

int check_ws(void* ws, size_t ws_bytes, size_t need) {
  if (!ws || ws_bytes < need) return GF_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return GF_ERR_INVALID_ARG;
  return GF_OK;
}

int cuda_status(cudaError_t e) { return e == cudaSuccess ? GF_OK : GF_ERR_CUDA; }

// Window heads [h_begin, h_begin+h_count) on `stream`.
int run_window(const Tuning& tn, const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d, int w,
               float scale, int dtype, int layout, int h_begin, int h_count, WsHeader* ws,
               cudaStream_t stream, bool two_sided = false) {
  if (h_count <= 0) return GF_OK;
  const int w_eff = w > N ? N : w;  // keys before token 0 (or after the last one) do not exist
  const int fwd = two_sided ? w_eff - 1 : 0;
  if (!tn.force_simt && gf::tc_window_supported(N, d, w_eff, dtype))
    return cuda_status(
        gf::launch_window_tc(q, k, v, o, B, H, N, d, w_eff, fwd, scale, layout, h_begin, h_count, ws, stream));
  return cuda_status(gf::launch_window_simt(q, k, v, o, B, N, d, w_eff, fwd, scale, dtype,
                                            gf::make_strides(layout, H, N, d), h_begin, h_count, stream));
}

// Feature map of the linear heads of one call: elu + 1 (W null), or positive random features under
// the projections W [h_count, d, d].  On the tensor-core path those are computed first, into the two
// feature tensors at the end of the workspace (feat_offset bytes in).
struct Phi {
  const void* W = nullptr;
  size_t feat_offset = 0;
};

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }
size_t feature_bytes(int B, int h_lin, int N, int d) { return align256((size_t)B * h_lin * N * d * 2); }

int check_phi(int phi, const void* W) {
  if (phi == GF_PHI_ELU1) return W == nullptr ? GF_OK : GF_ERR_INVALID_ARG;
  if (phi == GF_PHI_FAVOR_POS) return (W != nullptr && aligned16(W)) ? GF_OK : GF_ERR_INVALID_ARG;
  return GF_ERR_UNSUPPORTED;
}

int run_linear(const Tuning& tn, const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d, int dtype,
               int layout, int h_begin, int h_count, float* S_io, float* z_io, bool zero_init, int max_ctas,
               WsHeader* ws, cudaStream_t stream, bool shared = false, const Phi& phi = Phi(), int* first_grid = nullptr) {
  if (h_count <= 0) return GF_OK;
  if (!tn.force_simt && gf::tc_linear_supported(N, d, dtype)) {
    void *fq = nullptr, *fk = nullptr;
    if (phi.W != nullptr) {
      fq = reinterpret_cast<uint8_t*>(ws) + phi.feat_offset;
      fk = reinterpret_cast<uint8_t*>(fq) + feature_bytes(B, h_count, N, d);
      const int rc = cuda_status(gf::launch_favor_features_tc(q, k, phi.W, fq, fk, B, H, N, d, layout, h_begin,
                                                              h_count, ws, stream));
      if (rc != GF_OK) return rc;
    }
    return cuda_status(gf::launch_linear_tc(q, k, v, o, B, H, N, d, layout, h_begin, h_count, S_io, z_io,
                                            zero_init, tn.linear_split, max_ctas, ws, stream, shared, fq, fk, first_grid));
  }
  return cuda_status(gf::launch_linear_simt(q, k, v, o, B, N, d, dtype, gf::make_strides(layout, H, N, d),
                                            h_begin, h_count, S_io, z_io, zero_init, stream, false, phi.W));
}

// Zeroes the workspace header and, for a call that runs the tensor-core linear kernel on n_lin
// chains, the hand-over flags behind it: one memset, ahead of everything the call launches.
int clear_ws(const Tuning& tn, void* ws, cudaStream_t stream, int n_lin = 0, int N = 0, int d = 0, int dtype = GF_BF16) {
  size_t bytes = sizeof(WsHeader);
  if (n_lin > 0 && !tn.force_simt && gf::tc_linear_supported(N, d, dtype))
    bytes += gf::linear_tc_flag_bytes(n_lin, N, tn.linear_split);
  if (cudaMemsetAsync(ws, 0, bytes, stream) != cudaSuccess) return GF_ERR_CUDA;
  // the two test knobs travel in the header (all zero otherwise: nothing more to do)
  if (tn.wait_kcycles != 0 || tn.drop_flag != 0)
    return cuda_status(gf::launch_set_header((WsHeader*)ws, (unsigned int)tn.wait_kcycles, (unsigned int)tn.drop_flag, stream));
  return GF_OK;
}

size_t workspace_bytes(const Tuning& tn, int B, int H, int N, int d, int h_sparse, int dtype, int phi = GF_PHI_ELU1,
                       size_t* feat_offset = nullptr);

}  // namespace

extern "C" {

const char* gformer_status_string(int status) {
  switch (status) {
    case GF_OK: return "ok";
    case GF_ERR_INVALID_ARG: return "invalid argument";
    case GF_ERR_UNSUPPORTED: return "unsupported configuration";
    case GF_ERR_WORKSPACE: return "workspace missing or too small";
    case GF_ERR_CUDA: return "CUDA error";
    case GF_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

int gformer_version(void) { return 100; }

unsigned long long gformer_launch_count(void) { return gf::g_launches.load(std::memory_order_relaxed); }

int gformer_default_h_sparse(int H) {
  if (H < 1) return 0;
  int h0 = (int)floor(3.0 * H / 16.0 + 0.5);
  if (h0 < 1) h0 = 1;
  if (h0 > H) h0 = H;
  return h0;
}

int gformer_set_tuning(int key, int value) {
  switch (key) {
    case GF_TUNE_FORCE_SIMT:
      g_force_simt.store(value ? 1 : 0);
      return GF_OK;
    case GF_TUNE_WAIT_KCYCLES:
      if (value < 0) return GF_ERR_INVALID_ARG;
      g_wait_kcycles.store(value);
      return GF_OK;
    case GF_TUNE_TEST_DROP_FLAG:
      if (value < 0) return GF_ERR_INVALID_ARG;
      g_drop_flag.store(value);
      return GF_OK;
    case GF_TUNE_LINEAR_SPLIT:
      if (value < -1 || value > 4096) return GF_ERR_INVALID_ARG;
      g_linear_split.store(value);
      return GF_OK;
    case GF_TUNE_LINEAR_CTAS:
      if (value < 0 || value > 65535) return GF_ERR_INVALID_ARG;
      g_linear_ctas.store(value);
      return GF_OK;
    default:
      return GF_ERR_INVALID_ARG;
  }
}

int gformer_linear_plan(int chains, int N, int d, int ctas, int* segments, int* chunks_per_segment) {
  if (chains < 1 || N < 1 || ctas < 0 || segments == nullptr || chunks_per_segment == nullptr) return GF_ERR_INVALID_ARG;
  if (!gf::tc_linear_supported(N, d, GF_BF16)) return GF_ERR_UNSUPPORTED;
  gf::linear_tc_plan(chains, N, d, g_linear_split.load(), ctas, chunks_per_segment, segments);
  return GF_OK;
}

int gformer_linear_plan_parts(int chains, int N, int d, int ctas, int* whole_chains, int* segments,
                              int* chunks_per_segment) {
  if (chains < 1 || N < 1 || ctas < 0 || whole_chains == nullptr || segments == nullptr || chunks_per_segment == nullptr)
    return GF_ERR_INVALID_ARG;
  if (!gf::tc_linear_supported(N, d, GF_BF16)) return GF_ERR_UNSUPPORTED;
  gf::linear_tc_plan_parts(chains, N, d, g_linear_split.load(), ctas, whole_chains, chunks_per_segment, segments);
  return GF_OK;
}

size_t gformer_workspace_bytes(int B, int H, int N, int d, int w, int h_sparse, int dtype) {
  (void)w;
  return workspace_bytes(tuning_now(), B, H, N, d, h_sparse, dtype);
}

size_t gformer_workspace_bytes_phi(int B, int H, int N, int d, int w, int h_sparse, int dtype, int phi) {
  (void)w;
  return workspace_bytes(tuning_now(), B, H, N, d, h_sparse, dtype, phi);
}
}  // extern "C"

namespace {
size_t workspace_bytes(const Tuning& tn, int B, int H, int N, int d, int h_sparse, int dtype, int phi,
                       size_t* feat_offset) {
  size_t bytes = sizeof(WsHeader);
  if (feat_offset) *feat_offset = 0;
  if (B < 1 || H < 1 || N < 1) return bytes;
  if (h_sparse < 0) h_sparse = gformer_default_h_sparse(H);
  if (h_sparse > H) h_sparse = H;
  const int h_lin = H - h_sparse;
  if (h_lin > 0 && !tn.force_simt && gf::tc_linear_supported(N, d, dtype)) {
    // the causal kernel's hand-over scratch, or the bidirectional layer's segment sums: whichever is larger
    const size_t causal = gf::linear_tc_workspace_bytes(B * h_lin, N, d, tn.linear_split);
    const size_t self = gf::linear_self_workspace_bytes(B * h_lin, N, d);
    bytes += causal > self ? causal : self;
    if (phi == GF_PHI_FAVOR_POS) {  // the features of Q and K of the linear heads, behind everything else
      bytes = align256(bytes);
      if (feat_offset) *feat_offset = bytes;
      bytes += 2 * feature_bytes(B, h_lin, N, d);
    }
  }
  return bytes;
}
}  // namespace

extern "C" {

int gformer_last_device_status(void* ws, void* cuda_stream) {
  if (!ws) return GF_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  WsHeader hdr;
  if (cudaMemcpyAsync(&hdr, ws, sizeof(hdr), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return GF_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return GF_ERR_CUDA;
  return hdr.status == 0 ? GF_OK : GF_ERR_TIMEOUT;
}

int gformer_window_attn(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d, int w,
                        float scale, int dtype, int layout, void* ws, size_t ws_bytes, void* cuda_stream) {
  int rc = check_common(q, k, v, o, B, H, N, d, dtype, layout);
  if (rc != GF_OK) return rc;
  const Tuning tn = tuning_now();
  if (w < 1) return GF_ERR_INVALID_ARG;
  rc = check_ws(ws, ws_bytes, workspace_bytes(tn, B, H, N, d, H, dtype));
  if (rc != GF_OK) return rc;
  if (!(scale > 0.f)) scale = 1.0f / sqrtf((float)d);
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  rc = clear_ws(tn, ws, stream);
  if (rc != GF_OK) return rc;
  return run_window(tn, q, k, v, o, B, H, N, d, w, scale, dtype, layout, 0, H, (WsHeader*)ws, stream);
}

int gformer_window_attn_self(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d,
                             int w, float scale, int dtype, int layout, void* ws, size_t ws_bytes,
                             void* cuda_stream) {
  int rc = check_common(q, k, v, o, B, H, N, d, dtype, layout);
  if (rc != GF_OK) return rc;
  const Tuning tn = tuning_now();
  if (w < 1) return GF_ERR_INVALID_ARG;
  rc = check_ws(ws, ws_bytes, workspace_bytes(tn, B, H, N, d, H, dtype));
  if (rc != GF_OK) return rc;
  if (!(scale > 0.f)) scale = 1.0f / sqrtf((float)d);
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  rc = clear_ws(tn, ws, stream);
  if (rc != GF_OK) return rc;
  return run_window(tn, q, k, v, o, B, H, N, d, w, scale, dtype, layout, 0, H, (WsHeader*)ws, stream, true);
}

int gformer_hybrid_attn_self(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d,
                             int w, int h_sparse, float scale, int phi, int dtype, int layout, void* ws,
                             size_t ws_bytes, void* cuda_stream) {
  if (phi == GF_PHI_FAVOR_POS) return GF_ERR_INVALID_ARG;  // needs its projections: gformer_hybrid_attn_self_w
  return gformer_hybrid_attn_self_w(q, k, v, o, B, H, N, d, w, h_sparse, scale, phi, nullptr, dtype, layout, ws, ws_bytes,
                                    cuda_stream);
}

int gformer_hybrid_attn_self_w(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d,
                               int w, int h_sparse, float scale, int phi, const void* W, int dtype, int layout,
                               void* ws, size_t ws_bytes, void* cuda_stream) {
  int rc = check_common(q, k, v, o, B, H, N, d, dtype, layout);
  if (rc != GF_OK) return rc;
  const Tuning tn = tuning_now();
  if (w < 1) return GF_ERR_INVALID_ARG;
  if ((rc = check_phi(phi, W)) != GF_OK) return rc;
  size_t feat_offset = 0;
  if (h_sparse < 0) h_sparse = gformer_default_h_sparse(H);
  if (h_sparse > H) return GF_ERR_INVALID_ARG;
  rc = check_ws(ws, ws_bytes, workspace_bytes(tn, B, H, N, d, h_sparse, dtype, phi, &feat_offset));
  if (rc != GF_OK) return rc;
  if (!(scale > 0.f)) scale = 1.0f / sqrtf((float)d);
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  rc = clear_ws(tn, ws, stream);
  if (rc != GF_OK) return rc;
  const bool tc_linear = !tn.force_simt && gf::tc_linear_supported(N, d, dtype);
  // positive random features: computed first (on the stream the linear kernels run on), then read in
  // place of Q and K
  void *fq = nullptr, *fk = nullptr;
  if (W != nullptr && tc_linear && h_sparse < H) {
    fq = reinterpret_cast<uint8_t*>(ws) + feat_offset;
    fk = reinterpret_cast<uint8_t*>(fq) + feature_bytes(B, H - h_sparse, N, d);
  }
  if (h_sparse > 0 && h_sparse < H && tc_linear) {
    // Both head groups on tensor-core kernels: the three launches of the linear heads go to the
    // library's high-priority stream, the windowed heads to its side stream a few microseconds
    // later; their CTAs run while the small totals kernel has the device and in the tails of the
    // two big ones.  Forked from and joined back into the caller's stream.
    Fork* f = get_fork();
    if (f == nullptr) return GF_ERR_CUDA;
    std::unique_lock<std::mutex> enqueue_guard(f->enqueue);
    if (cudaEventRecord(f->fork, stream) != cudaSuccess) return GF_ERR_CUDA;
    if (cudaStreamWaitEvent(f->side, f->fork, 0) != cudaSuccess) return GF_ERR_CUDA;
    if (cudaStreamWaitEvent(f->first, f->fork, 0) != cudaSuccess) return GF_ERR_CUDA;
    if (fq != nullptr)
      rc = cuda_status(gf::launch_favor_features_tc(q, k, W, fq, fk, B, H, N, d, layout, h_sparse, H - h_sparse,
                                                    (WsHeader*)ws, f->first));
    int lin_grid = 0;
    if (rc == GF_OK)
      rc = cuda_status(gf::launch_linear_self_tc(q, k, v, o, B, H, N, d, layout, h_sparse, H - h_sparse, (WsHeader*)ws,
                                                 sizeof(WsHeader), f->first, fq, fk, &lin_grid));
    if (cudaEventRecord(f->join_first, f->first) != cudaSuccess) return GF_ERR_CUDA;
    if (cudaStreamWaitEvent(stream, f->join_first, 0) != cudaSuccess) return GF_ERR_CUDA;
    // the windowed heads start once the CTAs of the first linear kernel have all started
    int rc2 = (rc == GF_OK && lin_grid > 0)
                  ? cuda_status(gf::launch_wait_placed((WsHeader*)ws, (unsigned int)lin_grid, kPlacedWaitNs, f->side))
                  : GF_OK;
    if (rc2 == GF_OK)
      rc2 = run_window(tn, q, k, v, o, B, H, N, d, w, scale, dtype, layout, 0, h_sparse, (WsHeader*)ws, f->side, true);
    if (cudaEventRecord(f->join, f->side) != cudaSuccess) return GF_ERR_CUDA;
    if (cudaStreamWaitEvent(stream, f->join, 0) != cudaSuccess) return GF_ERR_CUDA;
    return rc != GF_OK ? rc : rc2;
  }
  rc = run_window(tn, q, k, v, o, B, H, N, d, w, scale, dtype, layout, 0, h_sparse, (WsHeader*)ws, stream, true);
  if (rc != GF_OK) return rc;
  if (h_sparse == H) return GF_OK;
  if (tc_linear) {
    if (fq != nullptr) {
      rc = cuda_status(gf::launch_favor_features_tc(q, k, W, fq, fk, B, H, N, d, layout, h_sparse, H - h_sparse,
                                                    (WsHeader*)ws, stream));
      if (rc != GF_OK) return rc;
    }
    return cuda_status(gf::launch_linear_self_tc(q, k, v, o, B, H, N, d, layout, h_sparse, H - h_sparse, (WsHeader*)ws,
                                                 sizeof(WsHeader), stream, fq, fk));
  }
  // fp32 storage (or the CUDA-core knob): token by token, a summing sweep and a readout sweep
  return cuda_status(gf::launch_linear_simt(q, k, v, o, B, N, d, dtype, gf::make_strides(layout, H, N, d), h_sparse,
                                            H - h_sparse, nullptr, nullptr, true, stream, true, W));
}

int gformer_causal_linear_attn(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d,
                               int phi, int chunk, float* S_io, float* z_io, int dtype, int layout, void* ws,
                               size_t ws_bytes, void* cuda_stream) {
  if (phi == GF_PHI_FAVOR_POS) return GF_ERR_INVALID_ARG;  // needs its projections: gformer_causal_linear_attn_w
  return gformer_causal_linear_attn_w(q, k, v, o, B, H, N, d, phi, nullptr, chunk, S_io, z_io, dtype, layout, ws,
                                      ws_bytes, cuda_stream);
}

int gformer_causal_linear_attn_w(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d,
                                 int phi, const void* W, int chunk, float* S_io, float* z_io, int dtype, int layout,
                                 void* ws, size_t ws_bytes, void* cuda_stream) {
  int rc = check_common(q, k, v, o, B, H, N, d, dtype, layout);
  if (rc != GF_OK) return rc;
  const Tuning tn = tuning_now();
  if ((rc = check_phi(phi, W)) != GF_OK) return rc;
  Phi fm;
  fm.W = W;
  if (chunk != 0 && chunk != 128) return chunk < 0 || chunk % 64 ? GF_ERR_INVALID_ARG : GF_ERR_UNSUPPORTED;
  if ((S_io == nullptr) != (z_io == nullptr)) return GF_ERR_INVALID_ARG;
  if (S_io && (!aligned16(S_io) || !aligned16(z_io))) return GF_ERR_INVALID_ARG;
  rc = check_ws(ws, ws_bytes, workspace_bytes(tn, B, H, N, d, 0, dtype, phi, &fm.feat_offset));
  if (rc != GF_OK) return rc;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  rc = clear_ws(tn, ws, stream, B * H, N, d, dtype);
  if (rc != GF_OK) return rc;
  return run_linear(tn, q, k, v, o, B, H, N, d, dtype, layout, 0, H, S_io, z_io, false, 0, (WsHeader*)ws, stream, false,
                    fm);
}

int gformer_hybrid_attn(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d, int w,
                        int h_sparse, float scale, int phi, int chunk, int dtype, int layout,
                        gf_decode_state* state_out, void* ws, size_t ws_bytes, void* cuda_stream) {
  if (phi == GF_PHI_FAVOR_POS) return GF_ERR_INVALID_ARG;  // needs its projections: gformer_hybrid_attn_w
  return gformer_hybrid_attn_w(q, k, v, o, B, H, N, d, w, h_sparse, scale, phi, nullptr, chunk, dtype, layout, state_out,
                               ws, ws_bytes, cuda_stream);
}

int gformer_hybrid_attn_w(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d, int w,
                          int h_sparse, float scale, int phi, const void* W, int chunk, int dtype, int layout,
                          gf_decode_state* state_out, void* ws, size_t ws_bytes, void* cuda_stream) {
  int rc = check_common(q, k, v, o, B, H, N, d, dtype, layout);
  if (rc != GF_OK) return rc;
  const Tuning tn = tuning_now();
  if (w < 1) return GF_ERR_INVALID_ARG;
  if ((rc = check_phi(phi, W)) != GF_OK) return rc;
  Phi fm;
  fm.W = W;
  if (chunk != 0 && chunk != 128) return chunk < 0 || chunk % 64 ? GF_ERR_INVALID_ARG : GF_ERR_UNSUPPORTED;
  if (h_sparse < 0) h_sparse = gformer_default_h_sparse(H);
  if (h_sparse > H) return GF_ERR_INVALID_ARG;
  const int h_lin = H - h_sparse;
  if (state_out) {
    gf_decode_state* s = state_out;
    if (s->B != B || s->H != H || s->d != d || s->w != w || s->h_sparse != h_sparse || s->dtype != dtype)
      return GF_ERR_INVALID_ARG;
    if (h_sparse > 0 && (!s->k_cache || !s->v_cache || !aligned16(s->k_cache) || !aligned16(s->v_cache)))
      return GF_ERR_INVALID_ARG;
    if (h_lin > 0 && (!s->S || !s->z || !aligned16(s->S) || !aligned16(s->z))) return GF_ERR_INVALID_ARG;
  }
  rc = check_ws(ws, ws_bytes, workspace_bytes(tn, B, H, N, d, h_sparse, dtype, phi, &fm.feat_offset));
  if (rc != GF_OK) return rc;
  if (!(scale > 0.f)) scale = 1.0f / sqrtf((float)d);
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  rc = clear_ws(tn, ws, stream, B * h_lin, N, d, dtype);
  if (rc != GF_OK) return rc;

  float* S_out = state_out ? state_out->S : nullptr;
  float* z_out = state_out ? state_out->z : nullptr;
  // The two head groups run side by side on two streams.  The persistent linear kernel holds one
  // CTA per SM it uses.  When it has work for every SM it still takes them all (measured on a
  // B200, leaving some to the windowed heads from the start was no faster and less steady), on a
  // stream of the highest priority; the windowed heads' short-lived CTAs then fill the SMs that
  // linear CTAs leave at different times towards the end.
  const bool both = h_sparse > 0 && h_lin > 0;
  int lin_ctas = 0;
  if (both && !tn.force_simt && gf::tc_linear_supported(N, d, dtype)) {
    int L = 0, G = 0, whole = 0, dev = 0, sms = 0;
    gf::linear_tc_plan_parts(B * h_lin, N, d, tn.linear_split, 0, &whole, &L, &G, true);
    if (whole > 0) G = 1;  // items of the first launch: the chains left whole
    if (gf::device_info(&dev, &sms) != cudaSuccess) return GF_ERR_CUDA;
    if ((long long)B * h_lin * G >= sms) {
      lin_ctas = (tn.linear_ctas > 0 && tn.linear_ctas < sms) ? tn.linear_ctas : sms;
    }
  }
  Fork* f = both ? get_fork() : nullptr;
  if (both && f == nullptr) return GF_ERR_CUDA;
  std::unique_lock<std::mutex> enqueue_guard;
  if (both) enqueue_guard = std::unique_lock<std::mutex>(f->enqueue);
  if (both) {
    // fork: the linear heads (the long serial chains) stay on the caller's stream, the
    // windowed heads go to the side stream; join before returning control to the stream.
    if (cudaEventRecord(f->fork, stream) != cudaSuccess) return GF_ERR_CUDA;
    if (cudaStreamWaitEvent(f->side, f->fork, 0) != cudaSuccess) return GF_ERR_CUDA;
  }
  // When the two kernels compete for SMs the linear one goes to a stream of the highest priority
  // (the caller's stream may well have the lowest, like the side stream).
  const bool lin_first = both && lin_ctas > 0;
  if (lin_first && cudaStreamWaitEvent(f->first, f->fork, 0) != cudaSuccess) return GF_ERR_CUDA;
  int lin_grid = 0;
  rc = run_linear(tn, q, k, v, o, B, H, N, d, dtype, layout, h_sparse, h_lin, S_out, z_out, true, lin_ctas,
                  (WsHeader*)ws, lin_first ? f->first : stream, both, fm, &lin_grid);
  if (lin_first) {
    if (cudaEventRecord(f->join_first, f->first) != cudaSuccess) return GF_ERR_CUDA;
    if (cudaStreamWaitEvent(stream, f->join_first, 0) != cudaSuccess) return GF_ERR_CUDA;
  }
  cudaStream_t wstream = both ? f->side : stream;
  // Both kernels become runnable at the fork.  CTAs of the persistent linear kernel wait for one
  // another and want every SM from the start, while a windowed-heads CTA that got onto an SM first
  // keeps it for many tiles: the side stream is held back until the linear kernel's CTAs have all
  // started (they count themselves in the workspace header), 20 microseconds at most.
  if (lin_first && rc == GF_OK && lin_grid > 0 &&
      cuda_status(gf::launch_wait_placed((WsHeader*)ws, (unsigned int)lin_grid, kPlacedWaitNs, wstream)) != GF_OK)
    return GF_ERR_CUDA;
  int rc2 = run_window(tn, q, k, v, o, B, H, N, d, w, scale, dtype, layout, 0, h_sparse, (WsHeader*)ws, wstream);
  if (rc2 == GF_OK && state_out && h_sparse > 0)
    rc2 = cuda_status(gf::launch_export_ring(k, v, state_out->k_cache, state_out->v_cache, B, N, d, w, dtype,
                                             gf::make_strides(layout, H, N, d), h_sparse, wstream));
  if (both) {
    if (cudaEventRecord(f->join, f->side) != cudaSuccess) return GF_ERR_CUDA;
    if (cudaStreamWaitEvent(stream, f->join, 0) != cudaSuccess) return GF_ERR_CUDA;
  }
  if (rc != GF_OK) return rc;
  if (rc2 != GF_OK) return rc2;
  if (state_out) state_out->t = N;
  return GF_OK;
}

static int decode_step_impl(const void* q, const void* k, const void* v, void* o, gf_decode_state* st,
                            long long* t_seq, float scale, int phi, const void* W, void* cuda_stream);

int gformer_decode_step(const void* q, const void* k, const void* v, void* o, gf_decode_state* st, float scale,
                        int phi, void* cuda_stream) {
  if (phi == GF_PHI_FAVOR_POS) return GF_ERR_INVALID_ARG;  // needs its projections: gformer_decode_step_w
  return decode_step_impl(q, k, v, o, st, nullptr, scale, phi, nullptr, cuda_stream);
}

int gformer_decode_step_w(const void* q, const void* k, const void* v, void* o, gf_decode_state* st, float scale,
                          int phi, const void* W, void* cuda_stream) {
  return decode_step_impl(q, k, v, o, st, nullptr, scale, phi, W, cuda_stream);
}

int gformer_decode_step_ragged(const void* q, const void* k, const void* v, void* o, gf_decode_state* st,
                               long long* t_seq, float scale, int phi, void* cuda_stream) {
  if (phi == GF_PHI_FAVOR_POS) return GF_ERR_INVALID_ARG;  // needs its projections: gformer_decode_step_ragged_w
  return gformer_decode_step_ragged_w(q, k, v, o, st, t_seq, scale, phi, nullptr, cuda_stream);
}

int gformer_decode_step_ragged_w(const void* q, const void* k, const void* v, void* o, gf_decode_state* st,
                                 long long* t_seq, float scale, int phi, const void* W, void* cuda_stream) {
  if (!t_seq || (reinterpret_cast<uintptr_t>(t_seq) & 7u) != 0) return GF_ERR_INVALID_ARG;
  if (st && st->H > 4096) return GF_ERR_UNSUPPORTED;  // the arrival count of a sequence's heads has 15 bits
  return decode_step_impl(q, k, v, o, st, t_seq, scale, phi, W, cuda_stream);
}

static int decode_step_impl(const void* q, const void* k, const void* v, void* o, gf_decode_state* st,
                            long long* t_seq, float scale, int phi, const void* W, void* cuda_stream) {
  if (!q || !k || !v || !o || !st) return GF_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return GF_ERR_INVALID_ARG;
  {
    const int rc = check_phi(phi, W);
    if (rc != GF_OK) return rc;
  }
  if (st->B < 1 || st->H < 1 || st->w < 1 || st->h_sparse < 0 || st->h_sparse > st->H || st->t < 0)
    return GF_ERR_INVALID_ARG;
  if (st->dtype != GF_F32 && st->dtype != GF_BF16) return GF_ERR_INVALID_ARG;
  if (st->d != 64 && st->d != 128) return GF_ERR_UNSUPPORTED;
  if (st->B > 65535) return GF_ERR_UNSUPPORTED;
  if ((size_t)st->w * sizeof(float) > 160 * 1024) return GF_ERR_UNSUPPORTED;
  if (st->h_sparse > 0 &&
      (!st->k_cache || !st->v_cache || !aligned16(st->k_cache) || !aligned16(st->v_cache)))
    return GF_ERR_INVALID_ARG;
  if (st->h_sparse < st->H && (!st->S || !st->z || !aligned16(st->S) || !aligned16(st->z)))
    return GF_ERR_INVALID_ARG;
  const size_t bytes = (size_t)st->B * st->H * st->d * elem_size(st->dtype);
  if (overlaps(o, q, bytes) || overlaps(o, k, bytes) || overlaps(o, v, bytes)) return GF_ERR_INVALID_ARG;
  if (!(scale > 0.f)) scale = 1.0f / sqrtf((float)st->d);
  cudaError_t e = gf::launch_decode_step(q, k, v, o, st->k_cache, st->v_cache, st->S, st->z, st->t, t_seq, st->B,
                                         st->H, st->d, st->w, st->h_sparse, scale, st->dtype,
                                         (cudaStream_t)cuda_stream, W);
  if (e != cudaSuccess) return GF_ERR_CUDA;
  if (t_seq == nullptr) st->t += 1;
  return GF_OK;
}

}  // extern "C"
