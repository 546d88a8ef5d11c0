// Chunked causal linear attention on the tensor cores (bf16 in, fp32 accumulate and state).
//
// Algorithm 1 regrouped 128 rows at a time (exactly equal by associativity).  For chunk c with
// Qc = phi(Q_c), Kc = phi(K_c):
//   P   = Qc Kc^T                       (MMA1)   masked to j <= i           -> Pm (bf16)
//   S_c = S_{c-1} + Kc^T V_c            (MMA4)   fp32 master copy lives in TMEM for the whole chain
//   O   = Qc Sb_{c-1}  (+)  Pm V_c      (MMA2, MMA3)  Sb = bf16 copy of S in shared memory
//   den = rowsum(Pm) + Qc z_{c-1},  z_c = z_{c-1} + colsum(Kc)      (fp32, CUDA cores)
//   out = O / den
// One CTA walks one (batch, head) chain.  Warp roles:
//   warp 0       TMA producer (raw Q, K, V tiles; K and V double buffered)
//   warp 1       MMA issuer
//   warps 2-5    "P group": masks/packs P in TMEM, converts S to bf16 for the next chunk's
//                readout, divides and stores O (one thread per row / TMEM lane)
//   warps 6-13   "phi(Q) group": applies phi to Q; the result goes to TMEM as the A operand of
//                MMA1/MMA2, together with the per-row dot product with z_{c-1}
//   warps 14-21  "phi(K) group": applies phi to K in place in shared memory and adds its column
//                sums to z
//   warp 22      stores O tiles (staged in the dead V buffer) with TMA
// TMEM (D=128): P 128 | O 128 | S 128 | phi(Q) 2 x 64 columns = 512.
// Every wait is bounded; on expiry the kernel records a status word and drains.
#include "common.cuh"
#include "sm100.cuh"

namespace gf {
namespace {

using namespace sm100;

constexpr int kThreads = 736;  // 23 warps, 88 registers each
constexpr float kLog2e = 1.4426950408889634f;

template <int D>
struct LinCfg {
  static constexpr int kTile = 128 * D * 2;  // one 128 x D bf16 tile
  static constexpr int kQ = 0;               // raw Q landing buffer
  static constexpr int kK = kTile;           // 2 stages
  static constexpr int kV = 3 * kTile;       // 2 stages
  static constexpr int kSb = 5 * kTile;      // bf16 copy of S, [D rows][D cols] in 64-column boxes
  static constexpr int kSbBytes = D * D * 2;
  static constexpr int kBytes = 5 * kTile + kSbBytes + 1024;
  static constexpr int kBoxBytes = 16384;    // one 128-row x 64-column box
  static constexpr int kSbBox = D * 128;     // one D-row x 64-column box of Sb
  // TMEM columns
  static constexpr uint32_t tP = 0, tO = 128, tS = 128 + D, tQ = 128 + 2 * D;  // tQ: 2 x D/2
  static constexpr uint32_t kTmemCols = 512;
};

struct LinParams {
  int N, h_begin, h_count;
  float* S_io;           // [B, h_count, D, D] or null
  float* z_io;           // [B, h_count, D] or null
  int zero_init;
  unsigned int* status;
};

struct LinBarriers {
  uint64_t q_full, q_land_free;
  uint64_t k_full[2], v_full[2], k_free[2], v_free[2];
  uint64_t qphi_full[2], kphi_full[2], qphi_free[2], qz_free[2];
  uint64_t p_full, s_full, o_full, mma2_done;
  uint64_t pm_full, s_loaded, sb_full, o_free, o_staged;
};

// Developer instrumentation (compiled only with -DGF_PROFILE): per-role time stamps of the first
// chunks of CTA (0,0), read back with gformer_debug_read_profile.
#ifdef GF_PROFILE
__device__ unsigned long long g_prof[4][64][8];
__device__ __forceinline__ void prof_stamp(int role, int c, int ev) {
  if (blockIdx.x == 0 && blockIdx.y == 0 && c < 64) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    g_prof[role][c][ev] = t;
  }
}
#define PROF(role, c, ev) prof_stamp(role, c, ev)
#else
#define PROF(role, c, ev)
#endif

// Named barrier over `n` threads that also ORs a predicate, so that a timed-out wait makes the
// whole group leave its loop together (nobody is left behind at a barrier).
__device__ __forceinline__ bool named_bar_or(int id, int n, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.or.pred p, %2, %3, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}\n"
      : "=r"(r)
      : "r"((uint32_t)pred), "r"(id), "r"(n)
      : "memory");
  return r != 0;
}

// phi(x) = elu(x) + 1 = max(x, 0) + exp(min(x, 0)) on two packed bf16 values (branch free; the
// result is needed in bf16 anyway).  log2(e) is split in two bf16 terms so that the exponent
// argument carries only the rounding of one bf16 product.
__device__ __forceinline__ uint32_t phi_bf16x2(uint32_t w) {
  const __nv_bfloat162 x = *reinterpret_cast<const __nv_bfloat162*>(&w);
  const __nv_bfloat162 zero = __float2bfloat162_rn(0.f);
  const __nv_bfloat162 l2e_hi = __float2bfloat162_rn(1.4453125f);
  const __nv_bfloat162 l2e_lo = __float2bfloat162_rn(kLog2e - 1.4453125f);
  const __nv_bfloat162 t = __hmin2(__hfma2(x, l2e_lo, __hmul2(x, l2e_hi)), zero);
  uint32_t e;  // native packed exponential (the header's h2exp2 goes through two fp32 ex2 + converts)
  asm("ex2.approx.ftz.bf16x2 %0, %1;" : "=r"(e) : "r"(*reinterpret_cast<const uint32_t*>(&t)));
  const __nv_bfloat162 f = __hadd2(__hmax2(x, zero), *reinterpret_cast<const __nv_bfloat162*>(&e));
  return *reinterpret_cast<const uint32_t*>(&f);
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
linear_tc_kernel(const __grid_constant__ CUtensorMap mq, const __grid_constant__ CUtensorMap mk,
                 const __grid_constant__ CUtensorMap mv, const __grid_constant__ CUtensorMap mo,
                 const LinParams p) {
  using C = LinCfg<D>;
  extern __shared__ uint8_t raw_smem[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(raw_smem) + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = sm + C::kQ;
  uint8_t* sK = sm + C::kK;
  uint8_t* sV = sm + C::kV;
  uint8_t* sSb = sm + C::kSb;
  __shared__ __align__(8) LinBarriers bar;
  __shared__ __align__(16) float zs[4][D];  // z before chunk c is zs[c & 3]
  __shared__ float qz[2][2][128];           // [chunk parity][column half][row]
  __shared__ int z_ready;                   // chunks whose column sums are in zs (monotonic)
  __shared__ uint32_t tmem_base_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int hl = blockIdx.x, b = blockIdx.y;
  const int h = p.h_begin + hl;
  const int nch = (p.N + 127) / 128;
  const long long sidx = (long long)b * p.h_count + hl;

  if (tid == 0) {
    mbar_init(&bar.q_full, 1);
    mbar_init(&bar.q_land_free, 8);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bar.k_full[s], 1);
      mbar_init(&bar.v_full[s], 1);
      mbar_init(&bar.k_free[s], 1);
      mbar_init(&bar.v_free[s], 1);
      mbar_init(&bar.qphi_full[s], 8);
      mbar_init(&bar.kphi_full[s], 8);
      mbar_init(&bar.qphi_free[s], 1);
      mbar_init(&bar.qz_free[s], 128);
    }
    mbar_init(&bar.p_full, 1);
    mbar_init(&bar.s_full, 1);
    mbar_init(&bar.o_full, 1);
    mbar_init(&bar.mma2_done, 1);
    mbar_init(&bar.pm_full, 128);
    mbar_init(&bar.s_loaded, 128);
    mbar_init(&bar.sb_full, 128);
    mbar_init(&bar.o_free, 128);
    mbar_init(&bar.o_staged, 128);
    z_ready = -1;
    mbar_fence_init();
    tma_prefetch_desc(&mq);
    tma_prefetch_desc(&mk);
    tma_prefetch_desc(&mv);
    tma_prefetch_desc(&mo);
  }
  if (warp == 1) {
    tmem_alloc(&tmem_base_s, C::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_base_s;

  if (warp == 0) {
    // ================================================================ TMA producer
    if (elect_one()) {
      for (int c = 0; c < nch; ++c) {
        const int s = c & 1, n0 = c * 128;
        if (c >= 2 && !mbar_wait(&bar.k_free[s], ((c >> 1) + 1) & 1, p.status, 101)) break;
        PROF(0, c, 1);
        mbar_arrive_expect_tx(&bar.k_full[s], C::kTile);
        for (int x = 0; x < D / 64; ++x)
          tma_load_4d(sK + s * C::kTile + x * C::kBoxBytes, &mk, &bar.k_full[s], x * 64, n0, h, b);
        if (c >= 1 && !mbar_wait(&bar.q_land_free, (c - 1) & 1, p.status, 100)) break;
        PROF(0, c, 0);
        mbar_arrive_expect_tx(&bar.q_full, C::kTile);
        for (int x = 0; x < D / 64; ++x) tma_load_4d(sQ + x * C::kBoxBytes, &mq, &bar.q_full, x * 64, n0, h, b);
        if (c >= 2 && !mbar_wait(&bar.v_free[s], ((c >> 1) + 1) & 1, p.status, 102)) break;
        PROF(0, c, 2);
        mbar_arrive_expect_tx(&bar.v_full[s], C::kTile);
        for (int x = 0; x < D / 64; ++x)
          tma_load_4d(sV + s * C::kTile + x * C::kBoxBytes, &mv, &bar.v_full[s], x * 64, n0, h, b);
      }
    }
  } else if (warp == 1) {
    // ================================================================ MMA issuer
    if (elect_one()) {
      constexpr uint32_t id_p = umma_idesc_bf16(128, 128, false, false);  // P  = Qc Kc^T
      constexpr uint32_t id_s = umma_idesc_bf16(128, D, true, true);      // S += Kc^T V
      constexpr uint32_t id_o = umma_idesc_bf16(128, D, false, true);     // O  = Qc Sb,  O += Pm V
      constexpr uint32_t kLboA = (D == 128) ? C::kBoxBytes : 0;           // D=64: rows 64..127 of S mirror 0..63
      for (int c = 0; c < nch; ++c) {
        const int s = c & 1;
        const uint32_t ph2 = (c >> 1) & 1;
        const uint32_t kbase = smem_u32(sK) + s * C::kTile, vbase = smem_u32(sV) + s * C::kTile;
        const uint32_t tq = tmem + C::tQ + s * (D / 2);
        if (!mbar_wait(&bar.qphi_full[s], ph2, p.status, 200)) break;
        if (!mbar_wait(&bar.kphi_full[s], ph2, p.status, 201)) break;
        PROF(1, c, 0);
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          umma_ts(tmem + C::tP, tq + ks * 8,
                  umma_smem_desc(kbase + (ks >> 2) * C::kBoxBytes + (ks & 3) * 32, 16, 1024), id_p, ks > 0);
        umma_commit(&bar.p_full);
        if (!mbar_wait(&bar.v_full[s], ph2, p.status, 202)) break;
        if (!mbar_wait(&bar.s_loaded, c & 1, p.status, 203)) break;
        PROF(1, c, 1);
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
          umma_ss(tmem + C::tS, umma_smem_desc(kbase + ks * 2048, kLboA, 1024),
                  umma_smem_desc(vbase + ks * 2048, C::kBoxBytes, 1024), id_s, true);
        umma_commit(&bar.s_full);
        umma_commit(&bar.k_free[s]);
        if (!mbar_wait(&bar.sb_full, c & 1, p.status, 204)) break;
        if (c >= 1 && !mbar_wait(&bar.o_free, (c - 1) & 1, p.status, 205)) break;
        PROF(1, c, 2);
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          umma_ts(tmem + C::tO, tq + ks * 8, umma_smem_desc(smem_u32(sSb) + ks * 2048, C::kSbBox, 1024), id_o,
                  ks > 0);
        umma_commit(&bar.mma2_done);
        umma_commit(&bar.qphi_free[s]);
        if (!mbar_wait(&bar.pm_full, c & 1, p.status, 206)) break;
        PROF(1, c, 3);
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
          umma_ts(tmem + C::tO, tmem + C::tP + ks * 8, umma_smem_desc(vbase + ks * 2048, C::kBoxBytes, 1024),
                  id_o, true);
        umma_commit(&bar.o_full);
      }
    }
  } else if (warp < 6) {
    // ================================================================ P group (one thread per row)
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const bool s_row = r < D;  // rows of S are feature indices a < D
    // ---- initial state: S (fp32) into TMEM, its bf16 copy into shared memory
    {
      const float* Sin = (p.S_io != nullptr && !p.zero_init) ? p.S_io + (sidx * D + r) * D : nullptr;
#pragma unroll
      for (int cc = 0; cc < D / 32; ++cc) {
        uint32_t v[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = (Sin != nullptr && s_row) ? __float_as_uint(Sin[cc * 32 + j]) : 0u;
        tmem_st32(tmem + C::tS + lane_off + cc * 32, v);
        if (s_row) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            uint4 val;
            val.x = pack_bf16(__uint_as_float(v[8 * g + 0]), __uint_as_float(v[8 * g + 1]));
            val.y = pack_bf16(__uint_as_float(v[8 * g + 2]), __uint_as_float(v[8 * g + 3]));
            val.z = pack_bf16(__uint_as_float(v[8 * g + 4]), __uint_as_float(v[8 * g + 5]));
            val.w = pack_bf16(__uint_as_float(v[8 * g + 6]), __uint_as_float(v[8 * g + 7]));
            const uint32_t col = (cc & 1) * 32 + g * 8;
            *reinterpret_cast<uint4*>(sSb + (cc >> 1) * C::kSbBox + swz128_offset(r, col)) = val;
          }
        }
      }
      tmem_wait_st();
      fence_proxy_async_smem();
      tc_fence_before_sync();
      mbar_arrive(&bar.s_loaded);
      mbar_arrive(&bar.sb_full);
    }
    for (int c = 0; c < nch; ++c) {
      const int s = c & 1;
      // ---- P: causal mask inside the chunk, row sum, bf16 back into TMEM
      if (!mbar_wait(&bar.qphi_full[s], (c >> 1) & 1, p.status, 300)) break;
      const float qzr = qz[s][0][r] + qz[s][1][r];
      mbar_arrive(&bar.qz_free[s]);
      if (!mbar_wait(&bar.p_full, c & 1, p.status, 301)) break;
      if (tid == 64) PROF(2, c, 0);
      tc_fence_after_sync();
      float rowsum = 0.f;
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        // 32-column block cc of this warp's rows [32 q, 32 q + 32): all kept left of the
        // diagonal block, all dropped right of it, triangular on it (warp-uniform choice)
        uint32_t pk[16];
        if (cc > quarter) {
#pragma unroll
          for (int j = 0; j < 16; ++j) pk[j] = 0u;
        } else {
          uint32_t v[32];
          tmem_ld32(tmem + C::tP + lane_off + cc * 32, v);
          tmem_wait_ld();
          const bool diag = (cc == quarter);
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float p0 = (!diag || 2 * j <= lane) ? __uint_as_float(v[2 * j]) : 0.f;
            const float p1 = (!diag || 2 * j + 1 <= lane) ? __uint_as_float(v[2 * j + 1]) : 0.f;
            rowsum += p0 + p1;
            pk[j] = pack_bf16(p0, p1);
          }
        }
        tmem_st16(tmem + C::tP + lane_off + cc * 16, pk);
      }
      const float den = rowsum + qzr;
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(&bar.pm_full);
      if (tid == 64) PROF(2, c, 1);
      // ---- S: the fp32 master stays in TMEM; once this chunk's readout has consumed the old bf16
      //      copy, stream the new one into shared memory for the next chunk
      if (!mbar_wait(&bar.s_full, c & 1, p.status, 302)) break;
      if (tid == 64) PROF(2, c, 2);
      if (!mbar_wait(&bar.mma2_done, c & 1, p.status, 303)) break;
      if (tid == 64) PROF(2, c, 3);
      tc_fence_after_sync();
      const bool last = (c == nch - 1);
#pragma unroll
      for (int cc = 0; cc < D / 32; ++cc) {
        uint32_t v[32];
        tmem_ld32(tmem + C::tS + lane_off + cc * 32, v);
        tmem_wait_ld();
        if (s_row) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            uint4 val;
            val.x = pack_bf16(__uint_as_float(v[8 * g + 0]), __uint_as_float(v[8 * g + 1]));
            val.y = pack_bf16(__uint_as_float(v[8 * g + 2]), __uint_as_float(v[8 * g + 3]));
            val.z = pack_bf16(__uint_as_float(v[8 * g + 4]), __uint_as_float(v[8 * g + 5]));
            val.w = pack_bf16(__uint_as_float(v[8 * g + 6]), __uint_as_float(v[8 * g + 7]));
            *reinterpret_cast<uint4*>(sSb + (cc >> 1) * C::kSbBox + swz128_offset(r, (cc & 1) * 32 + g * 8)) = val;
          }
          if (last && p.S_io != nullptr) {
            float* dst = p.S_io + (sidx * D + r) * D + cc * 32;
#pragma unroll
            for (int j = 0; j < 32; j += 4)
              *reinterpret_cast<float4*>(dst + j) =
                  make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]), __uint_as_float(v[j + 2]),
                              __uint_as_float(v[j + 3]));
          }
        }
      }
      tc_fence_before_sync();
      mbar_arrive(&bar.s_loaded);
      fence_proxy_async_smem();
      mbar_arrive(&bar.sb_full);
      if (tid == 64) PROF(2, c, 5);
      // ---- O: divide by the denominator, bf16, stage for the TMA store
      if (!mbar_wait(&bar.o_full, c & 1, p.status, 304)) break;
      if (tid == 64) PROF(2, c, 6);
      tc_fence_after_sync();
      const float inv = 1.f / den;
      uint8_t* stage = sV + s * C::kTile;  // V_c is dead once MMA3 of this chunk has completed
#pragma unroll
      for (int cc = 0; cc < D / 32; ++cc) {
        uint32_t v[32];
        tmem_ld32(tmem + C::tO + lane_off + cc * 32, v);
        tmem_wait_ld();
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          uint4 val;
          val.x = pack_bf16(__uint_as_float(v[8 * g + 0]) * inv, __uint_as_float(v[8 * g + 1]) * inv);
          val.y = pack_bf16(__uint_as_float(v[8 * g + 2]) * inv, __uint_as_float(v[8 * g + 3]) * inv);
          val.z = pack_bf16(__uint_as_float(v[8 * g + 4]) * inv, __uint_as_float(v[8 * g + 5]) * inv);
          val.w = pack_bf16(__uint_as_float(v[8 * g + 6]) * inv, __uint_as_float(v[8 * g + 7]) * inv);
          *reinterpret_cast<uint4*>(stage + (cc >> 1) * C::kBoxBytes + swz128_offset(r, (cc & 1) * 32 + g * 8)) = val;
        }
      }
      tc_fence_before_sync();
      mbar_arrive(&bar.o_free);
      fence_proxy_async_smem();
      mbar_arrive(&bar.o_staged);
      if (tid == 64) PROF(2, c, 7);
    }
  } else if (warp < 14) {
    // ================================================================ phi(Q) group (8 warps)
    const int quarter = warp & 3;         // TMEM lane quarter of this warp
    const int half = (warp - 6) >> 2;     // which half of the head dimension this warp handles
    const int r = quarter * 32 + lane;    // Q row
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    constexpr int kChunksPerHalf = D / 16;  // 16-byte chunks of one row handled per thread
    for (int c = 0; c < nch; ++c) {
      const int s = c & 1;
      bool ok = mbar_wait(&bar.q_full, c & 1, p.status, 400);
      if (tid == 192) PROF(3, c, 0);
      if (ok && c >= 2) {
        ok = mbar_wait(&bar.qphi_free[s], ((c >> 1) + 1) & 1, p.status, 401) &&  // phi(Q) buffer s is free
             mbar_wait(&bar.qz_free[s], ((c >> 1) + 1) & 1, p.status, 402);      // qz[s] of chunk c-2 was read
      }
      // z before this chunk = column sums of chunks < c, published by the phi(K) group
      if (ok) {
        const long long t0 = clock64();
        while (*reinterpret_cast<volatile int*>(&z_ready) < c) {
          if (clock64() - t0 > 4000000000LL) {
            if (atomicCAS(p.status, 0u, 1u) == 0u) p.status[1] = 403;
            ok = false;
            break;
          }
          __nanosleep(32);
        }
        __threadfence_block();
      }
      if (tid == 192) PROF(3, c, 1);
      tc_fence_after_sync();
      if (ok) {
        uint32_t pk[kChunksPerHalf * 4];
        float dot[2] = {0.f, 0.f};
        const float* zc = zs[c & 3];
#pragma unroll
        for (int g = 0; g < kChunksPerHalf; ++g) {
          const int gl = half * kChunksPerHalf + g;  // logical 16-byte chunk within the row (8 columns)
          const int box = gl >> 3, cin = gl & 7;
          const uint4 rawv = *reinterpret_cast<const uint4*>(sQ + box * C::kBoxBytes + r * 128 + ((cin ^ (r & 7)) << 4));
          const uint32_t w4[4] = {rawv.x, rawv.y, rawv.z, rawv.w};
          const float4 za = *reinterpret_cast<const float4*>(zc + gl * 8);
          const float4 zb = *reinterpret_cast<const float4*>(zc + gl * 8 + 4);
          const float zv[8] = {za.x, za.y, za.z, za.w, zb.x, zb.y, zb.z, zb.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const uint32_t pkv = phi_bf16x2(w4[e]);
            pk[g * 4 + e] = pkv;
            // the dot product uses the rounded values the tensor core will see
            dot[e & 1] = fmaf(bf16_lo(pkv), zv[2 * e], dot[e & 1]);
            dot[e & 1] = fmaf(bf16_hi(pkv), zv[2 * e + 1], dot[e & 1]);
          }
        }
        qz[s][half][r] = dot[0] + dot[1];
        if constexpr (D == 128) {
          uint32_t(&pk32)[32] = *reinterpret_cast<uint32_t(*)[32]>(pk);
          tmem_st32(tmem + C::tQ + s * (D / 2) + lane_off + half * 32, pk32);
        } else {
          tmem_st16(tmem + C::tQ + s * (D / 2) + lane_off + half * 16, pk);
        }
        tmem_wait_st();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(&bar.qphi_full[s]);
          mbar_arrive(&bar.q_land_free);
        }
      }
      if (tid == 192) PROF(3, c, 2);
      if (__any_sync(0xffffffffu, !ok)) break;
    }
  } else if (warp < 22) {
    // ================================================================ phi(K) group (8 warps)
    const int tt = tid - 14 * 32;  // 0..255
    if (tt < D) zs[0][tt] = (p.z_io != nullptr && !p.zero_init) ? p.z_io[sidx * D + tt] : 0.f;
    asm volatile("bar.sync 3, 256;" ::: "memory");
    if (tt == 0) {
      __threadfence_block();
      *reinterpret_cast<volatile int*>(&z_ready) = 0;  // zs[0] holds the initial z
    }
    for (int c = 0; c < nch; ++c) {
      const int s = c & 1;
      const bool ok = mbar_wait(&bar.k_full[s], (c >> 1) & 1, p.status, 410);
      if (tt == 0) PROF(3, c, 4);
      if (ok && tt < 2 * D) {
        const int cc = tt >> 4;  // logical 16-byte column chunk 0 .. D/8-1
        const int box = cc >> 3, cin = cc & 7;
        uint8_t* kb = sK + s * C::kTile + box * C::kBoxBytes;
        float cs[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) cs[e] = 0.f;
        // all loads first, then branch-free arithmetic, then all stores (the tile is updated in place)
        uint4 rawv[8];
#pragma unroll
        for (int k8 = 0; k8 < 8; ++k8) {
          const int row = (tt & 15) + 16 * k8;
          rawv[k8] = *reinterpret_cast<const uint4*>(kb + row * 128 + ((cin ^ (row & 7)) << 4));
        }
#pragma unroll
        for (int k8 = 0; k8 < 8; ++k8) {
          const int row = (tt & 15) + 16 * k8;
          const uint32_t keep = ((c * 128 + row) < p.N) ? 0xffffffffu : 0u;  // rows past N must not enter S, z
          uint32_t w4[4] = {rawv[k8].x, rawv[k8].y, rawv[k8].z, rawv[k8].w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            w4[e] = phi_bf16x2(w4[e]) & keep;
            cs[2 * e] += bf16_lo(w4[e]);
            cs[2 * e + 1] += bf16_hi(w4[e]);
          }
          rawv[k8] = make_uint4(w4[0], w4[1], w4[2], w4[3]);
        }
#pragma unroll
        for (int k8 = 0; k8 < 8; ++k8) {
          const int row = (tt & 15) + 16 * k8;
          *reinterpret_cast<uint4*>(kb + row * 128 + ((cin ^ (row & 7)) << 4)) = rawv[k8];
        }
        fence_proxy_async_smem();
#pragma unroll
        for (int e = 0; e < 8; ++e) {
#pragma unroll
          for (int off = 8; off > 0; off >>= 1) cs[e] += __shfl_xor_sync(0xffffffffu, cs[e], off);
        }
        if ((tt & 15) == 0) {
#pragma unroll
          for (int e = 0; e < 8; ++e) zs[(c + 1) & 3][cc * 8 + e] = zs[c & 3][cc * 8 + e] + cs[e];
        }
      }
      __syncwarp();
      if (ok && lane == 0) mbar_arrive(&bar.kphi_full[s]);
      if (tt == 0) PROF(3, c, 5);
      if (named_bar_or(3, 256, !ok)) break;
      if (tt == 0) {
        __threadfence_block();
        *reinterpret_cast<volatile int*>(&z_ready) = c + 1;
      }
    }
    if (p.z_io != nullptr && tt < D) p.z_io[sidx * D + tt] = zs[nch & 3][tt];
  } else {
    // ================================================================ O store warp
    if (elect_one()) {
      for (int c = 0; c < nch; ++c) {
        const int s = c & 1;
        if (!mbar_wait(&bar.o_staged, c & 1, p.status, 500)) break;
        for (int x = 0; x < D / 64; ++x)
          tma_store_4d(&mo, sV + s * C::kTile + x * C::kBoxBytes, x * 64, c * 128, h, b);
        tma_store_commit();
        tma_store_wait_read<0>();
        mbar_arrive(&bar.v_free[s]);  // the staging buffer may take V of chunk c+2
      }
      tma_store_wait_all<0>();
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, C::kTmemCols);
}

}  // namespace

#ifdef GF_PROFILE
extern "C" int gformer_debug_read_profile(unsigned long long* host_dst) {
  return (int)cudaMemcpyFromSymbol(host_dst, g_prof, sizeof(g_prof));
}
#endif

bool tc_linear_supported(int N, int d, int dtype) {
  (void)N;
  return dtype == GF_BF16 && (d == 64 || d == 128);
}

cudaError_t launch_linear_tc(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d,
                             int layout, int h_begin, int h_count, float* S_io, float* z_io, bool zero_init,
                             int split, WsHeader* ws, cudaStream_t stream) {
  (void)split;
  if (h_count <= 0) return cudaSuccess;
  CUtensorMap mq, mk, mv, mo;
  if (!make_qkv_tensor_map(&mq, q, B, H, N, d, layout, 128) || !make_qkv_tensor_map(&mk, k, B, H, N, d, layout, 128) ||
      !make_qkv_tensor_map(&mv, v, B, H, N, d, layout, 128) || !make_qkv_tensor_map(&mo, o, B, H, N, d, layout, 128))
    return cudaErrorInvalidValue;
  LinParams p;
  p.N = N;
  p.h_begin = h_begin;
  p.h_count = h_count;
  p.S_io = S_io;
  p.z_io = z_io;
  p.zero_init = zero_init ? 1 : 0;
  p.status = &ws->status;
  dim3 grid(h_count, B);
  cudaError_t e;
  if (d == 64) {
    auto kern = linear_tc_kernel<64>;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, LinCfg<64>::kBytes);
    if (e != cudaSuccess) return e;
    kern<<<grid, kThreads, LinCfg<64>::kBytes, stream>>>(mq, mk, mv, mo, p);
  } else {
    auto kern = linear_tc_kernel<128>;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, LinCfg<128>::kBytes);
    if (e != cudaSuccess) return e;
    kern<<<grid, kThreads, LinCfg<128>::kBytes, stream>>>(mq, mk, mv, mo, p);
  }
  note_launch();
  return cudaGetLastError();
}

}  // namespace gf
