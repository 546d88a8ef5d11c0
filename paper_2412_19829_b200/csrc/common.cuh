// Shared declarations of the libgformer CUDA sources (host-side launch interfaces and a
// few device helpers).  Not part of the public ABI.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gformer.h"

namespace gf {

// Element strides of a logical [B, H, N, d] tensor (innermost stride is 1).
struct Strides {
  long long b, h, n;
};

inline Strides make_strides(int layout, int H, int N, int d) {
  Strides s;
  if (layout == GF_BNHD) {
    s.b = (long long)N * H * d;
    s.n = (long long)H * d;
    s.h = d;
  } else {
    s.b = (long long)H * N * d;
    s.h = (long long)N * d;
    s.n = d;
  }
  return s;
}

// Layout of the first bytes of the caller's workspace.
struct WsHeader {
  unsigned int status;   // 0 = fine, else a code written by a kernel whose bounded wait expired
  unsigned int where;    // which wait gave up (diagnostic)
  unsigned int ticket;   // work counter of the persistent kernels
  unsigned int wait_kcycles;  // limit of every bounded wait in units of 1024 cycles; 0 = default (about 2 s)
  unsigned int drop_flag;     // failure injection for tests: the linear kernel skips the flag of segment n - 1
  unsigned int placed;        // CTAs of the call's linear-attention kernels that have started (see launch_wait_placed)
  unsigned int pad[58];
};
static_assert(sizeof(WsHeader) == 256, "workspace header is 256 bytes");

// Counts kernel launches (reported by gformer_launch_count).
void note_launch(int n = 1);

// ---- SIMT (CUDA-core, fp32 arithmetic) path: any w, d in {64,128}, f32 or bf16 storage.
// Heads [h_begin, h_begin + h_count) of the [B, H, N, d] tensors are processed.
// fwd: keys after the query it may see: 0 = the causal window, w - 1 = the two-sided window |i - j| < w.
cudaError_t launch_window_simt(const void* q, const void* k, const void* v, void* o, int B, int N, int d,
                               int w, int fwd, float scale, int dtype, Strides st, int h_begin, int h_count,
                               cudaStream_t stream);
// S_io/z_io: [B, h_count, d, d] / [B, h_count, d] or null.  zero_init: ignore their contents on entry.
// global_sum: the unmasked linear attention of the bidirectional layer (sum over all tokens, then readout).
cudaError_t launch_linear_simt(const void* q, const void* k, const void* v, void* o, int B, int N, int d,
                               int dtype, Strides st, int h_begin, int h_count, float* S_io, float* z_io,
                               bool zero_init, cudaStream_t stream, bool global_sum = false,
                               const void* W = nullptr /* [h_count, d, d] storage dtype: positive random features */);
cudaError_t launch_export_ring(const void* k, const void* v, void* k_cache, void* v_cache, int B, int N, int d,
                               int w, int dtype, Strides st, int h_sparse, cudaStream_t stream);
// t_seq == nullptr: every sequence is at position t; else sequence b is at t_seq[b] (device array,
// negative = idle slot, otherwise below 2^48) and the kernel itself moves the positions on.
cudaError_t launch_decode_step(const void* q, const void* k, const void* v, void* o, void* k_cache,
                               void* v_cache, float* S, float* z, long long t, long long* t_seq, int B, int H,
                               int d, int w, int h_sparse, float scale, int dtype, cudaStream_t stream,
                               const void* W = nullptr /* [H - h_sparse, d, d] storage dtype */);

// Writes the two test knobs into a workspace header that has just been cleared.
cudaError_t launch_set_header(WsHeader* ws, unsigned int wait_kcycles, unsigned int drop_flag, cudaStream_t stream);

// One tiny CTA that returns once `target` CTAs of the call's linear-attention kernel have started
// (WsHeader::placed), or after max_ns nanoseconds whichever comes first: holds back the work queued
// behind it in its stream without occupying an SM's shared memory or tensor memory.  Never an error:
// when the limit ends the wait, the work behind it simply starts.
cudaError_t launch_wait_placed(WsHeader* ws, unsigned int target, unsigned int max_ns, cudaStream_t stream);

// The current device and its SM count (asked of the driver once per device).
cudaError_t device_info(int* dev, int* sms);
// cudaFuncAttributeMaxDynamicSharedMemorySize of a kernel, set once per kernel and device.
cudaError_t ensure_dynamic_smem(const void* kernel, int dev, int bytes);

// ---- tensor-core (tcgen05 / TMEM / TMA) path: bf16 storage, d in {64,128}.
bool tc_window_supported(int N, int d, int w, int dtype);
bool tc_linear_supported(int N, int d, int dtype);
cudaError_t launch_window_tc(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d,
                             int w, int fwd, float scale, int layout, int h_begin, int h_count, WsHeader* ws,
                             cudaStream_t stream);
// Global (unmasked) linear attention of the bidirectional layer, heads [h_begin, h_begin + h_count):
// three launches (segment sums, totals, readout); its scratch starts scratch_offset bytes into ws.
size_t linear_self_workspace_bytes(int nchains, int N, int d);
cudaError_t launch_linear_self_tc(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d,
                                  int layout, int h_begin, int h_count, WsHeader* ws, size_t scratch_offset,
                                  cudaStream_t stream, const void* fq = nullptr, const void* fk = nullptr,
                                  int* first_grid = nullptr /* CTAs of the first launch */);
// Segmentation used by the tensor-core linear kernel (split: 0 = automatic, else chunks per segment;
// ctas: CTAs the kernel will run with, 0 = one per SM of a B200) and the scratch it needs beyond
// the workspace header (sized for the largest segment count the plan may pick for any ctas).
void linear_tc_plan(int nchains, int N, int d, int split, int ctas, int* chunks_per_segment, int* segments_per_chain);
// The same plan with its two parts named: the first *whole_chains chains are left whole, the others cut
// (with somewhat more chains than CTAs the full rounds go whole and the leftover chains are cut, in a
// second launch); *whole_chains = nchains and one segment per chain when nothing is cut.
// shared: other kernels run beside this one and fill the SMs a thin round of whole chains leaves idle.
void linear_tc_plan_parts(int nchains, int N, int d, int split, int ctas, int* whole_chains, int* chunks_per_segment,
                          int* segments_per_chain, bool shared = false);
size_t linear_tc_workspace_bytes(int nchains, int N, int d, int split);
// Bytes at the start of that scratch (right after the workspace header) that must be zero when the
// kernel starts: the hand-over flags.  The caller clears them (together with the header).
size_t linear_tc_flag_bytes(int nchains, int N, int split);
cudaError_t launch_linear_tc(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d,
                             int layout, int h_begin, int h_count, float* S_io, float* z_io, bool zero_init,
                             int split, int max_ctas, WsHeader* ws, cudaStream_t stream, bool shared = false,
                             const void* fq = nullptr, const void* fk = nullptr,
                             int* first_grid = nullptr /* CTAs of the first launch */);
// Positive random features phi_W of Q and K of heads [h_begin, h_begin + h_count) (bf16 storage) into the
// contiguous bf16 tensors fq, fk [B, h_count, N, d]; W: [h_count, d, d] bf16, row a of a head's matrix is
// its projection vector w_a.  With fq, fk given, the two linear-attention launchers read them in place
// of Q and K and leave their own feature map out.
cudaError_t launch_favor_features_tc(const void* q, const void* k, const void* W, void* fq, void* fk, int B, int H,
                                     int N, int d, int layout, int h_begin, int h_count, WsHeader* ws,
                                     cudaStream_t stream);

// ---- device helpers
// Cycles a bounded wait may take; `status` points at the first word of the workspace header.
__device__ __forceinline__ long long wait_limit_cycles(const unsigned int* status) {
  const unsigned int kc = reinterpret_cast<const volatile unsigned int*>(status)[3];
  return kc ? (long long)kc * 1024 : 4000000000LL;
}

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) {
  return __float2bfloat16_rn(x);
}

// phi(x) = elu(x) + 1 (Sec. II-B).
__device__ __forceinline__ float phi_elu1(float x) { return x > 0.f ? x + 1.f : expf(x); }

}  // namespace gf
