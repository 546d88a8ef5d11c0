// Positive random features of the linear heads (Sec. III-A / III-C: "positive orthogonal random
// features"; the formula is the cited Performer paper's):
//     phi_W(x)[a] = exp(<w_a, x> - |x|^2 / 2) / sqrt(d),   a = 0 .. d-1,
// for every token of Q and of K of the linear heads, written as bf16 tensors [B, heads, N, d] that the
// chunked linear-attention kernels then read in place of Q and K (with their own feature map
// switched off).  A positive factor common to all features of one query cancels in
// o_i = phi(q_i)^T S / <phi(q_i), z>, so the query features are taken relative to the row's largest
// projection, exp(<w_a, q> - max_a <w_a, q>) (no |q|^2 / 2, no 1 / sqrt(d)): they then lie in (0, 1]
// and their products with the state stay inside the range of fp32 however small the key features
// are.  The key features (and with them the state S, z) are the definition's.
//
// One CTA = 128 tokens of one (batch, head) of Q or of K: the token tile X (128 x d) and the head's
// projection W (d x d, row a = w_a) come by TMA; one tcgen05.mma group computes Y = X W^T
// (M = 128, N = d, K = d, both operands K-major from shared memory) into TMEM; 128 threads, one per
// token, add up |x|^2 from the tile in shared memory, take the exponentials and write the features
// over the tile, which a TMA store ships (rows past the end of the sequence are clipped).
#include "common.cuh"
#include "sm100.cuh"

namespace gf {
namespace {

using namespace sm100;

constexpr int kFavorThreads = 192;  // warp 0: TMA, warp 1: MMA, warps 2..5: one thread per token
constexpr float kLog2eF = 1.4426950408889634f;

struct FavorParams {
  int h_begin, h_count;  // heads [h_begin, h_begin + h_count) of the input tensors
  unsigned int* status;
};

template <int D>
__global__ void __launch_bounds__(kFavorThreads)
favor_tc_kernel(const __grid_constant__ CUtensorMap mxq, const __grid_constant__ CUtensorMap mxk,
                const __grid_constant__ CUtensorMap mw, const __grid_constant__ CUtensorMap mfq,
                const __grid_constant__ CUtensorMap mfk, const FavorParams p) {
  constexpr int kTile = 128 * D * 2, kW = D * D * 2;
  extern __shared__ __align__(1024) uint8_t raw_smem[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(raw_smem) + 1023) & ~(uintptr_t)1023);
  uint8_t* sX = sm;
  uint8_t* sW = sm + kTile;
  __shared__ __align__(8) uint64_t full, done;
  __shared__ uint32_t tmem_base_s;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // (the (batch, head) index is the x coordinate of the grid, which has the range for it)
  const int i0 = blockIdx.y * 128;
  const int hl = blockIdx.x % p.h_count, b = blockIdx.x / p.h_count;
  const bool is_k = blockIdx.z != 0;
  const CUtensorMap* mx = is_k ? &mxk : &mxq;
  const CUtensorMap* mf = is_k ? &mfk : &mfq;
  if (tid == 0) {
    mbar_init(&full, 1);
    mbar_init(&done, 1);
    mbar_fence_init();
    tma_prefetch_desc(mx);
    tma_prefetch_desc(&mw);
    tma_prefetch_desc(mf);
  }
  if (warp == 1) {
    tmem_alloc(&tmem_base_s, D);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_base_s;
  if (warp == 0) {
    if (elect_one()) {
      mbar_arrive_expect_tx(&full, kTile + kW);
      for (int c = 0; c < D / 64; ++c) {
        tma_load_4d(sX + c * 16384, mx, &full, c * 64, i0, p.h_begin + hl, b);
        tma_load_4d(sW + c * (D * 128), &mw, &full, c * 64, 0, hl, 0);
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      constexpr uint32_t idesc = umma_idesc_bf16(128, D, false, false);
      if (mbar_wait(&full, 0, p.status, 900)) {
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          umma_ss(tmem, umma_smem_desc(smem_u32(sX) + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024),
                  umma_smem_desc(smem_u32(sW) + (ks >> 2) * (D * 128) + (ks & 3) * 32, 16, 1024), idesc, ks > 0);
        umma_commit(&done);
      }
    }
  } else {
    const int quarter = warp & 3;  // TMEM lane quarter this warp may touch
    const int r = quarter * 32 + lane;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const bool ok = mbar_wait(&done, 0, p.status, 901);  // the products are done: X is no longer read by the tensor core
    tc_fence_after_sync();
    if (ok) {
      // |x|^2 of this thread's token from the tile (128-byte swizzle: 16-byte chunks)
      float n2 = 0.f;
#pragma unroll
      for (int c8 = 0; c8 < D / 8; ++c8) {
        const uint4 v4 = *reinterpret_cast<const uint4*>(sX + (c8 >> 3) * 16384 + swz128_offset(r, (c8 & 7) * 8));
        const uint32_t w4[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w4[e]));
          n2 = fmaf(f.x, f.x, n2);
          n2 = fmaf(f.y, f.y, n2);
        }
      }
      // keys: exp(y - n2 / 2) / sqrt(d) = 2^((y - n2 / 2) log2(e) - log2(d) / 2);
      // queries: exp(y - max_a y) (the row's factor cancels in the output)
      float shift = -0.5f * n2 * kLog2eF - 0.5f * log2f((float)D);
      if (!is_k) {
        float mx = -INFINITY;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t y[32];
          tmem_ld32(tmem + lane_off + c * 32, y);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) mx = fmaxf(mx, __uint_as_float(y[e]));
        }
        shift = -mx * kLog2eF;
      }
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t y[32];
        tmem_ld32(tmem + lane_off + c * 32, y);
        tmem_wait_ld();
        uint8_t* box = sX + (c >> 1) * 16384;
#pragma unroll
        for (int g = 0; g < 4; ++g) {  // 4 chunks of 8 features
          float f[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) f[e] = exp2f(fmaf(__uint_as_float(y[8 * g + e]), kLog2eF, shift));
          uint4 val;
          val.x = pack_bf16(f[0], f[1]);
          val.y = pack_bf16(f[2], f[3]);
          val.z = pack_bf16(f[4], f[5]);
          val.w = pack_bf16(f[6], f[7]);
          *reinterpret_cast<uint4*>(box + swz128_offset(r, (c & 1) * 32 + g * 8)) = val;
        }
      }
      tc_fence_before_sync();
      fence_proxy_async_smem();
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (ok && warp == 2 && elect_one()) {
      for (int c = 0; c < D / 64; ++c) tma_store_4d(mf, sX + c * 16384, c * 64, i0, p.h_begin + hl, b);
      tma_store_commit();
      tma_store_wait_all<0>();
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, D);
}

}  // namespace

cudaError_t launch_favor_features_tc(const void* q, const void* k, const void* W, void* fq, void* fk, int B, int H,
                                     int N, int d, int layout, int h_begin, int h_count, WsHeader* ws,
                                     cudaStream_t stream) {
  if (h_count <= 0) return cudaSuccess;
  CUtensorMap mxq, mxk, mw, mfq, mfk;
  if (!make_qkv_tensor_map(&mxq, q, B, H, N, d, layout, 128) || !make_qkv_tensor_map(&mxk, k, B, H, N, d, layout, 128) ||
      !make_feature_tensor_map(&mfq, fq, B, H, N, d, h_begin, h_count, 128) ||
      !make_feature_tensor_map(&mfk, fk, B, H, N, d, h_begin, h_count, 128) ||
      !make_qkv_tensor_map(&mw, W, 1, h_count, d, d, GF_BHND, d))  // [1, heads, d features, d inputs]: box of d rows
    return cudaErrorInvalidValue;
  FavorParams p;
  p.h_begin = h_begin;
  p.h_count = h_count;
  p.status = &ws->status;
  const long long rows = (long long)B * h_count, tiles = ((long long)N + 127) / 128;
  if (rows > 0x7fffffffLL || tiles > 65535) return cudaErrorInvalidValue;  // (tiles: more than 8 million tokens)
  dim3 grid((unsigned)rows, (unsigned)tiles, 2);
  auto launch = [&](auto kern, int smem) -> cudaError_t {
    int dev = 0, sms = 0;
    cudaError_t err = device_info(&dev, &sms);
    if (err == cudaSuccess) err = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), dev, smem);
    if (err != cudaSuccess) return err;
    kern<<<grid, kFavorThreads, smem, stream>>>(mxq, mxk, mw, mfq, mfk, p);
    note_launch();
    return cudaGetLastError();
  };
  return d == 64 ? launch(favor_tc_kernel<64>, 128 * 64 * 2 + 64 * 64 * 2 + 1024)
                 : launch(favor_tc_kernel<128>, 128 * 128 * 2 + 128 * 128 * 2 + 1024);
}

}  // namespace gf
