// Global (unmasked) linear attention on the tensor cores: the linear heads of the bidirectional
// ("self") layer.  Sec. II-B without the causal mask:
//   S = sum_j phi(K_j) (x) V_j,  z = sum_j phi(K_j)   over the whole sequence,
//   out_i = phi(Q_i)^T S / (phi(Q_i) . z).
// Three launches, bf16 in, fp32 accumulate:
//   reduce   a chain is cut into segments; a CTA walks a segment's 128-row chunks: K and V tiles by
//            TMA, phi(K) in place in shared memory (16 warps), [S | z] += phi(K)^T [V | 1] as one
//            tcgen05.mma per 16 keys with N = D + 16 (V's B operand is followed by a constant box
//            whose column 0 is all ones, so z is column D of the accumulator); the segment's sum
//            goes from TMEM to a scratch slot of its own.
//   sum      adds the segments' slots of a chain in a fixed order (CUDA cores): deterministic totals.
//   readout  a CTA loads a chain's totals once per item as the bf16 B operand [Sb | hi(z) lo(z)],
//            then per chunk: Q tile by TMA, phi(Q) into TMEM (8 warps), one product with
//            N = D + 16 leaves the numerators and, in columns D and D + 1, the denominator split
//            in two; 4 epilogue warps divide, pack and stage the tile for a TMA store.
// Every wait is bounded; on expiry the kernel records a status word and drains.
#include "common.cuh"
#include "sm100.cuh"

namespace gf {
namespace {

using namespace sm100;

constexpr float kLog2eS = 1.4426950408889634f;
constexpr int kBox = 16384;  // one 128-row x 64-column bf16 box (what one TMA copy moves)

// phi(x) = elu(x) + 1 = max(x, 0) + exp(min(x, 0)) on two packed bf16 values (branch free); log2(e)
// is split in two bf16 terms so that the exponent argument carries the rounding of one product.
__device__ __forceinline__ uint32_t phi2(uint32_t w) {
  const __nv_bfloat162 x = *reinterpret_cast<const __nv_bfloat162*>(&w);
  const __nv_bfloat162 zero = __float2bfloat162_rn(0.f);
  const __nv_bfloat162 l2e_hi = __float2bfloat162_rn(1.4453125f);
  const __nv_bfloat162 l2e_lo = __float2bfloat162_rn(kLog2eS - 1.4453125f);
  const __nv_bfloat162 t = __hmin2(__hfma2(x, l2e_lo, __hmul2(x, l2e_hi)), zero);
  uint32_t e;
  asm("ex2.approx.ftz.bf16x2 %0, %1;" : "=r"(e) : "r"(*reinterpret_cast<const uint32_t*>(&t)));
  const __nv_bfloat162 f = __hadd2(__hmax2(x, zero), *reinterpret_cast<const __nv_bfloat162*>(&e));
  return *reinterpret_cast<const uint32_t*>(&f);
}

// kId: the tensors read as Q and K already hold features: the feature map here is the identity.
template <bool kId>
__device__ __forceinline__ uint32_t phi_sel(uint32_t w) {
  if constexpr (kId) return w;
  else return phi2(w);
}

struct SelfParams {
  int N, nch, h_begin, h_count, nchains;
  int G, seg_base, seg_rem, nitems;  // segments per chain (balanced lengths), nchains * G
  float* partial;                    // [nitems][D*D + D]: a segment's sums (S row-major [feature][column], then z)
  float* total;                      // [nchains][D*D + D]
  unsigned int* status;
};

struct SelfItem {
  int chain, g, b, h, c_begin, nC;
};

__device__ __forceinline__ SelfItem self_item(const SelfParams& p, int item) {
  SelfItem it;
  it.chain = item / p.G;
  it.g = item - it.chain * p.G;
  it.b = it.chain / p.h_count;
  it.h = p.h_begin + (it.chain - it.b * p.h_count);
  it.c_begin = it.g * p.seg_base + (it.g < p.seg_rem ? it.g : p.seg_rem);
  it.nC = p.seg_base + (it.g < p.seg_rem ? 1 : 0);
  return it;
}

// ------------------------------------------------------------------------------------ reduce
template <int D>
struct RedCfg {
  static constexpr int kTile = 128 * D * 2;
  // V | ones: one constant box serves every V slot, a box distance past the slot's last box:
  //   D = 128:  V0a . V1a V0b V1b . ONES   (slot 0: distance 3 boxes, slot 1: 2; two boxes unused)
  //   D = 64:   V0 V1 V2 V3 ONES           (slot s: distance 4 - s)
  static constexpr int kVSlots = (D == 128) ? 2 : 4;
  __host__ __device__ static constexpr int v_off(int s) { return (D == 128) ? (s ? 2 : 0) * kBox : s * kBox; }
  __host__ __device__ static constexpr int v_lbo(int s) { return (D == 128) ? (s ? 2 : 3) * kBox : (4 - s) * kBox; }
  static constexpr int kOnes = (D == 128) ? 6 * kBox : 4 * kBox;
  static constexpr int kK = kOnes + kBox;  // three K slots, contiguous
  static constexpr int kKSlots = 3;
  static constexpr int kBytes = kK + kKSlots * kTile + 1024;
  static constexpr int kAcc = D + 16;  // accumulator columns: S, then z in column D
  static constexpr int kThreads = 22 * 32;
};

template <int D, bool kId>
__global__ void __launch_bounds__(RedCfg<D>::kThreads, 1)
linear_self_reduce_kernel(const __grid_constant__ CUtensorMap mk, const __grid_constant__ CUtensorMap mv,
                          const SelfParams p) {
  using C = RedCfg<D>;
  constexpr int VS = C::kVSlots, KS = C::kKSlots;
  extern __shared__ uint8_t raw_smem[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(raw_smem) + 1023) & ~(uintptr_t)1023);
  uint8_t* sK = sm + C::kK;
  uint8_t* sOnes = sm + C::kOnes;
  __shared__ __align__(8) uint64_t k_full[KS], kphi[KS], k_free[KS], v_full[4], v_free[4], acc_done[2], acc_free[2];
  __shared__ uint32_t tmem_base_s;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    atomicAdd(&p.status[5], 1u);  // WsHeader::placed: this CTA has an SM
    for (int i = 0; i < KS; ++i) {
      mbar_init(&k_full[i], 1);
      mbar_init(&kphi[i], 16);
      mbar_init(&k_free[i], 1);
    }
    for (int i = 0; i < 4; ++i) {
      mbar_init(&v_full[i], 1);
      mbar_init(&v_free[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&acc_done[i], 1);
      mbar_init(&acc_free[i], 128);
    }
    mbar_fence_init();
    tma_prefetch_desc(&mk);
    tma_prefetch_desc(&mv);
  }
  if (warp == 1) {
    tmem_alloc(&tmem_base_s, 512);
    tmem_relinquish();
  } else if (warp >= 2) {
    // constant ones box: column 0 of every key row is 1 (128B swizzle: the row's first 16-byte
    // chunk sits at position row & 7), all else 0
    for (int i = tid - 64; i < kBox / 4; i += C::kThreads - 64) {
      const int row = i >> 5, w = i & 31;
      reinterpret_cast<uint32_t*>(sOnes)[i] = (w == ((row & 7) << 2)) ? 0x00003F80u : 0u;
    }
    fence_proxy_async_smem();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_base_s;

  // Every role walks the same items and keeps the same running counters: nk = K tiles so far
  // (slot nk % KS, phase nk / KS), nv likewise for V, na = items so far (accumulator na & 1).
  if (warp == 0) {
    if (elect_one()) {
      uint32_t nk = 0, nv = 0;
      bool ok = true;
      const uint64_t pol = l2_policy_evict_first();
      for (int item = blockIdx.x; item < p.nitems && ok; item += gridDim.x) {
        const SelfItem it = self_item(p, item);
        for (int j = 0; j < it.nC && ok; ++j) {
          const int n0 = (it.c_begin + j) * 128;
          const uint32_t sk = nk % KS, sv = nv % VS;
          if (nk >= KS && !mbar_wait(&k_free[sk], ((nk / KS) + 1) & 1, p.status, 700)) { ok = false; break; }
          mbar_arrive_expect_tx(&k_full[sk], C::kTile);
          for (int x = 0; x < D / 64; ++x)
            tma_load_4d_hint(sK + sk * C::kTile + x * kBox, &mk, &k_full[sk], x * 64, n0, it.h, it.b, pol);
          ++nk;
          if (nv >= VS && !mbar_wait(&v_free[sv], ((nv / VS) + 1) & 1, p.status, 701)) { ok = false; break; }
          mbar_arrive_expect_tx(&v_full[sv], C::kTile);
          for (int x = 0; x < D / 64; ++x)
            tma_load_4d_hint(sm + C::v_off(sv) + x * C::v_lbo(sv), &mv, &v_full[sv], x * 64, n0, it.h, it.b, pol);
          ++nv;
        }
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      constexpr uint32_t id_s = umma_idesc_bf16(128, C::kAcc, true, true);  // [S | z] += Kc^T [V | 1]
      constexpr uint32_t kLboA = (D == 128) ? kBox : 0;                     // D=64: rows 64..127 mirror 0..63
      uint32_t nk = 0, nv = 0, na = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < p.nitems && ok; item += gridDim.x, ++na) {
        const SelfItem it = self_item(p, item);
        const uint32_t acc = tmem + (na & 1) * C::kAcc;
        // the accumulator's previous sum has left TMEM
        if (na >= 2 && !mbar_wait(&acc_free[na & 1], ((na >> 1) + 1) & 1, p.status, 710)) break;
        for (int j = 0; j < it.nC; ++j) {
          const uint32_t sk = nk % KS, sv = nv % VS;
          if (!mbar_wait(&kphi[sk], (nk / KS) & 1, p.status, 711) ||
              !mbar_wait(&v_full[sv], (nv / VS) & 1, p.status, 712)) {
            ok = false;
            break;
          }
          tc_fence_after_sync();
          const uint32_t kbase = smem_u32(sK) + sk * C::kTile, vbase = smem_u32(sm) + C::v_off(sv);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            umma_ss(acc, umma_smem_desc(kbase + ks * 2048, kLboA, 1024),
                    umma_smem_desc(vbase + ks * 2048, C::v_lbo(sv), 1024), id_s, (j > 0) || (ks > 0));
          umma_commit(&k_free[sk]);
          umma_commit(&v_free[sv]);
          ++nk;
          ++nv;
        }
        if (!ok) break;
        umma_commit(&acc_done[na & 1]);
      }
    }
  } else if (warp < 6) {
    // drain: one thread per feature row writes the segment's sums to its scratch slot
    const int quarter = warp & 3, r = quarter * 32 + lane;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    uint32_t na = 0;
    for (int item = blockIdx.x; item < p.nitems; item += gridDim.x, ++na) {
      if (!mbar_wait(&acc_done[na & 1], (na >> 1) & 1, p.status, 720)) break;
      tc_fence_after_sync();
      const uint32_t acc = tmem + (na & 1) * C::kAcc + lane_off;
      float* dst = p.partial + (long long)item * (D * D + D);
#pragma unroll 1
      for (int cc = 0; cc < D / 32; ++cc) {
        uint32_t v[32];
        tmem_ld32(acc + cc * 32, v);
        tmem_wait_ld();
        if (r < D) {
#pragma unroll
          for (int jj = 0; jj < 32; jj += 4)
            *reinterpret_cast<float4*>(dst + (long long)r * D + cc * 32 + jj) =
                make_float4(__uint_as_float(v[jj]), __uint_as_float(v[jj + 1]), __uint_as_float(v[jj + 2]),
                            __uint_as_float(v[jj + 3]));
        }
      }
      const uint32_t zc = tmem_ld1(acc + D);
      tmem_wait_ld();
      if (r < D) dst[D * D + r] = __uint_as_float(zc);
      tc_fence_before_sync();
      mbar_arrive(&acc_free[na & 1]);
    }
  } else {
    // phi on the K tiles, in place: two groups of 8 warps, 64 rows each; thread = (16-byte column
    // chunk, row within sixteen), four rows sixteen apart
    const bool grp = warp >= 14;
    const int tt = grp ? tid - 14 * 32 : tid - 6 * 32;
    const int cc = tt >> 4, l16 = tt & 15;
    uint32_t nk = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < p.nitems && ok; item += gridDim.x) {
      const SelfItem it = self_item(p, item);
      for (int j = 0; j < it.nC; ++j) {
        const uint32_t sk = nk % KS;
        ok = ok && mbar_wait(&k_full[sk], (nk / KS) & 1, p.status, 730);
        if (ok && tt < 2 * D) {
          uint8_t* kb = sK + sk * C::kTile + (cc >> 3) * kBox;
          const int cin = cc & 7, n_valid = p.N - (it.c_begin + j) * 128;
          uint4 rawv[4];
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int row = l16 + 16 * ((grp ? 0 : 4) + k);
            rawv[k] = *reinterpret_cast<const uint4*>(kb + row * 128 + ((cin ^ (row & 7)) << 4));
          }
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int row = l16 + 16 * ((grp ? 0 : 4) + k);
            const uint32_t keep = (row < n_valid) ? 0xffffffffu : 0u;  // rows past the end contribute nothing
            rawv[k].x = phi_sel<kId>(rawv[k].x) & keep;
            rawv[k].y = phi_sel<kId>(rawv[k].y) & keep;
            rawv[k].z = phi_sel<kId>(rawv[k].z) & keep;
            rawv[k].w = phi_sel<kId>(rawv[k].w) & keep;
            *reinterpret_cast<uint4*>(kb + row * 128 + ((cin ^ (row & 7)) << 4)) = rawv[k];
          }
          fence_proxy_async_smem();
        }
        __syncwarp();
        if (ok && lane == 0) mbar_arrive(&kphi[sk]);
        ++nk;
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------------------------ sum
// total[chain] = sum over the chain's segments, in segment order (deterministic).
__global__ void linear_self_sum_kernel(const float* __restrict__ partial, float* __restrict__ total, int G,
                                       int state_floats) {
  const int chain = blockIdx.y;
  const int i = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i >= state_floats) return;
  const float* src = partial + (long long)chain * G * state_floats + i;
  float4 acc = *reinterpret_cast<const float4*>(src);
  for (int g = 1; g < G; ++g) {
    const float4 x = *reinterpret_cast<const float4*>(src + (long long)g * state_floats);
    acc.x += x.x;
    acc.y += x.y;
    acc.z += x.z;
    acc.w += x.w;
  }
  *reinterpret_cast<float4*>(total + (long long)chain * state_floats + i) = acc;
}

// ------------------------------------------------------------------------------------ readout
template <int D>
struct OutCfg {
  static constexpr int kTile = 128 * D * 2;
  static constexpr int kSbBox = D * 128;  // one D-row x 64-column box of the B operand
  static constexpr int kQ = 0;            // two raw Q tiles
  static constexpr int kSb = 2 * kTile;   // bf16 totals [D rows][D columns] in 64-column boxes ...
  static constexpr int kZb = kSb + D * D * 2;  // ... followed by one more box: columns 0, 1 = hi(z), lo(z)
  static constexpr int kStage = kZb + kSbBox;  // two output tiles staged for the TMA store
  static constexpr int kBytes = kStage + 2 * kTile + 1024;
  static constexpr int kAcc = D + 16;
  static constexpr uint32_t tQ = 0, tO = D;  // phi(Q): 2 x D/2 columns; O | den: 2 x (D + 16)
  static constexpr int kThreads = 15 * 32;
};

template <int D, bool kId>
__global__ void __launch_bounds__(OutCfg<D>::kThreads, 1)
linear_self_readout_kernel(const __grid_constant__ CUtensorMap mq, const __grid_constant__ CUtensorMap mo,
                           const SelfParams p) {
  using C = OutCfg<D>;
  extern __shared__ uint8_t raw_smem[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(raw_smem) + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = sm + C::kQ;
  uint8_t* sSb = sm + C::kSb;
  uint8_t* sZb = sm + C::kZb;
  uint8_t* sStage = sm + C::kStage;
  __shared__ __align__(8) uint64_t q_full[2], q_free[2], qphi_full[2], tq_free[2], o_full[2], o_free[2], sb_ready,
      o_staged[2], stage_free[2];
  __shared__ uint32_t tmem_base_s;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&q_full[i], 1);
      mbar_init(&q_free[i], 8);
      mbar_init(&qphi_full[i], 8);
      mbar_init(&tq_free[i], 1);
      mbar_init(&o_full[i], 1);
      mbar_init(&o_free[i], 128);
    }
    mbar_init(&sb_ready, 128);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&o_staged[i], 128);
      mbar_init(&stage_free[i], 1);
    }
    mbar_fence_init();
    tma_prefetch_desc(&mq);
    tma_prefetch_desc(&mo);
  }
  if (warp == 1) {
    tmem_alloc(&tmem_base_s, 512);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_base_s;

  // Running counters shared by all roles: nq = chunks so far (Q slot, phi(Q) slot and O buffer
  // nq & 1, phase nq >> 1; staging buffer phase nq), ni = items so far.
  if (warp == 0) {
    if (elect_one()) {
      uint32_t nq = 0;
      bool ok = true;
      const uint64_t pol = l2_policy_evict_first();
      for (int item = blockIdx.x; item < p.nitems && ok; item += gridDim.x) {
        const SelfItem it = self_item(p, item);
        for (int j = 0; j < it.nC; ++j, ++nq) {
          const uint32_t s = nq & 1;
          if (nq >= 2 && !mbar_wait(&q_free[s], ((nq >> 1) + 1) & 1, p.status, 800)) { ok = false; break; }
          mbar_arrive_expect_tx(&q_full[s], C::kTile);
          for (int x = 0; x < D / 64; ++x)
            tma_load_4d_hint(sQ + s * C::kTile + x * kBox, &mq, &q_full[s], x * 64, (it.c_begin + j) * 128, it.h, it.b,
                             pol);
        }
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      constexpr uint32_t id_o = umma_idesc_bf16(128, C::kAcc, false, true);  // [O | den] = Qc [Sb | Zb]
      uint32_t nq = 0, ni = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < p.nitems && ok; item += gridDim.x, ++ni) {
        const SelfItem it = self_item(p, item);
        if (!mbar_wait(&sb_ready, ni & 1, p.status, 810)) break;  // this item's totals are in shared memory
        for (int j = 0; j < it.nC; ++j, ++nq) {
          const uint32_t s = nq & 1;
          if (!mbar_wait(&qphi_full[s], (nq >> 1) & 1, p.status, 811) ||
              (nq >= 2 && !mbar_wait(&o_free[s], ((nq >> 1) + 1) & 1, p.status, 812))) {
            ok = false;
            break;
          }
          tc_fence_after_sync();
          const uint32_t tq = tmem + C::tQ + s * (D / 2), to = tmem + C::tO + s * C::kAcc;
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks)
            umma_ts(to, tq + ks * 8, umma_smem_desc(smem_u32(sSb) + ks * 2048, C::kSbBox, 1024), id_o, ks > 0);
          umma_commit(&o_full[s]);
          umma_commit(&tq_free[s]);
        }
      }
    }
  } else if (warp < 6) {
    // epilogue warps (one thread per row): load the chain's totals as the B operand at the start of an
    // item; per chunk divide the numerators by the denominator and stage the tile
    const int quarter = warp & 3, r = quarter * 32 + lane;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const bool s_row = r < D;
    uint32_t nq = 0, ni = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < p.nitems && ok; item += gridDim.x, ++ni) {
      const SelfItem it = self_item(p, item);
      // (the previous item's last product has completed: its o_full was seen below)
      if (s_row) {
        const float* src = p.total + (long long)it.chain * (D * D + D);
#pragma unroll 1
        for (int cc = 0; cc < D / 32; ++cc) {
          float4 in[8];
#pragma unroll
          for (int jj = 0; jj < 8; ++jj) in[jj] = __ldcg(reinterpret_cast<const float4*>(src + (long long)r * D + cc * 32) + jj);
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            uint4 val;
            val.x = pack_bf16(in[2 * g].x, in[2 * g].y);
            val.y = pack_bf16(in[2 * g].z, in[2 * g].w);
            val.z = pack_bf16(in[2 * g + 1].x, in[2 * g + 1].y);
            val.w = pack_bf16(in[2 * g + 1].z, in[2 * g + 1].w);
            *reinterpret_cast<uint4*>(sSb + (cc >> 1) * C::kSbBox + swz128_offset(r, (cc & 1) * 32 + g * 8)) = val;
          }
        }
        const float z = __ldcg(src + D * D + r);
        const float hi = __bfloat162float(__float2bfloat16_rn(z));
        // row r of the extra box: columns 0, 1 = hi(z), lo(z); the other 14 columns the product reads are zero
        uint4 zrow[2] = {make_uint4(pack_bf16(hi, z - hi), 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u)};
        *reinterpret_cast<uint4*>(sZb + swz128_offset(r, 0)) = zrow[0];
        *reinterpret_cast<uint4*>(sZb + swz128_offset(r, 8)) = zrow[1];
      }
      fence_proxy_async_smem();
      mbar_arrive(&sb_ready);
      for (int j = 0; j < it.nC; ++j, ++nq) {
        const uint32_t s = nq & 1;
        if (!mbar_wait(&o_full[s], (nq >> 1) & 1, p.status, 820) ||
            (nq >= 2 && !mbar_wait(&stage_free[s], ((nq >> 1) + 1) & 1, p.status, 821))) {
          ok = false;
          break;
        }
        tc_fence_after_sync();
        const uint32_t to = tmem + C::tO + s * C::kAcc + lane_off;
        uint32_t den_hi, den_lo;
        tmem_ld2(to + D, den_hi, den_lo);
        tmem_wait_ld();
        const float inv = 1.f / (__uint_as_float(den_hi) + __uint_as_float(den_lo));
#pragma unroll 1
        for (int cc = 0; cc < D / 32; ++cc) {
          uint32_t v[32];
          tmem_ld32(to + cc * 32, v);
          tmem_wait_ld();
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            uint4 val;
            val.x = pack_bf16(__uint_as_float(v[8 * g + 0]) * inv, __uint_as_float(v[8 * g + 1]) * inv);
            val.y = pack_bf16(__uint_as_float(v[8 * g + 2]) * inv, __uint_as_float(v[8 * g + 3]) * inv);
            val.z = pack_bf16(__uint_as_float(v[8 * g + 4]) * inv, __uint_as_float(v[8 * g + 5]) * inv);
            val.w = pack_bf16(__uint_as_float(v[8 * g + 6]) * inv, __uint_as_float(v[8 * g + 7]) * inv);
            *reinterpret_cast<uint4*>(sStage + s * C::kTile + (cc >> 1) * kBox + swz128_offset(r, (cc & 1) * 32 + g * 8)) = val;
          }
        }
        tc_fence_before_sync();
        mbar_arrive(&o_free[s]);
        fence_proxy_async_smem();
        mbar_arrive(&o_staged[s]);
      }
    }
  } else if (warp < 14) {
    // phi(Q): thread = (row, half of the head dimension); the result is the A operand in TMEM
    const int quarter = warp & 3, half = ((warp - 6) >> 2) & 1, r = quarter * 32 + lane;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    constexpr int kChunks = D / 16;  // 16-byte chunks of one row half
    uint32_t nq = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < p.nitems && ok; item += gridDim.x) {
      const SelfItem it = self_item(p, item);
      for (int j = 0; j < it.nC && ok; ++j, ++nq) {
        const uint32_t s = nq & 1;
        ok = mbar_wait(&q_full[s], (nq >> 1) & 1, p.status, 830);
        uint32_t pk[kChunks * 4];
        if (ok) {
#pragma unroll
          for (int g = 0; g < kChunks; ++g) {
            const int gl = half * kChunks + g, box = gl >> 3, cin = gl & 7;
            const uint4 rawv = *reinterpret_cast<const uint4*>(sQ + s * C::kTile + box * kBox + r * 128 +
                                                               ((cin ^ (r & 7)) << 4));
            pk[g * 4 + 0] = rawv.x;
            pk[g * 4 + 1] = rawv.y;
            pk[g * 4 + 2] = rawv.z;
            pk[g * 4 + 3] = rawv.w;
          }
        }
        // the buffer goes back to the TMA engine: these reads (generic proxy) must be ordered before its
        // next write (async proxy), which a barrier arrival alone does not do
        __threadfence_block();
        fence_proxy_async_smem();
        __syncwarp();
        if (ok && lane == 0) mbar_arrive(&q_free[s]);  // this warp has its part of the raw tile in registers
        if (ok) {
#pragma unroll
          for (int w = 0; w < kChunks * 4; ++w) pk[w] = phi_sel<kId>(pk[w]);
          if (nq >= 2) ok = mbar_wait(&tq_free[s], ((nq >> 1) + 1) & 1, p.status, 831);
        }
        tc_fence_after_sync();
        if (ok) {
          if constexpr (D == 128) {
            uint32_t(&pk32)[32] = *reinterpret_cast<uint32_t(*)[32]>(pk);
            tmem_st32(tmem + C::tQ + s * (D / 2) + lane_off + half * 32, pk32);
          } else {
            tmem_st16(tmem + C::tQ + s * (D / 2) + lane_off + half * 16, pk);
          }
          tmem_wait_st();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&qphi_full[s]);
        }
        ok = !__any_sync(0xffffffffu, !ok);
      }
    }
  } else {
    // TMA stores of the staged output tiles
    if (elect_one()) {
      uint32_t nq = 0;
      bool ok = true;
      const uint64_t pol = l2_policy_evict_first();
      for (int item = blockIdx.x; item < p.nitems && ok; item += gridDim.x) {
        const SelfItem it = self_item(p, item);
        for (int j = 0; j < it.nC; ++j, ++nq) {
          const uint32_t s = nq & 1;
          if (!mbar_wait(&o_staged[s], (nq >> 1) & 1, p.status, 840)) { ok = false; break; }
          for (int x = 0; x < D / 64; ++x)
            tma_store_4d_hint(&mo, sStage + s * C::kTile + x * kBox, x * 64, (it.c_begin + j) * 128, it.h, it.b, pol);
          tma_store_commit();
          // the other buffer's store (the previous chunk's) has read its tile: hand that buffer back
          if (nq >= 1) {
            tma_store_wait_read<1>();
            mbar_arrive(&stage_free[s ^ 1]);
          }
        }
      }
      tma_store_wait_all<0>();
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 512);
}

// Segments per chain.  CTAs take items (segments) round-robin, so a launch lasts ceil(items / CTAs)
// rounds of one item each: among the segment counts that keep segments at least four chunks long
// (and the scratch within 64 slots per chain, more when the chains are few), take the one with the least rounds x (chunks of the
// longest segment + about one chunk of fixed cost per item).  The plan must not depend on the
// device that is current when the workspace size is asked for: it assumes the 148 SMs of a B200.
int self_segments(int nchains, int nch) {
  constexpr int kPlanSMs = 148;
  int g_max = (nch + 3) / 4;
  int cap = (2 * kPlanSMs + nchains - 1) / nchains;  // few chains: as many segments as fill two rounds
  if (cap < 64) cap = 64;
  if (g_max > cap) g_max = cap;
  int best_g = 1;
  long long best = -1;
  for (int g = 1; g <= g_max; ++g) {
    const long long rounds = ((long long)nchains * g + kPlanSMs - 1) / kPlanSMs;
    const long long cost = rounds * ((nch + g - 1) / g + 1);
    if (best < 0 || cost < best) {
      best = cost;
      best_g = g;
    }
  }
  return best_g;
}

}  // namespace

size_t linear_self_workspace_bytes(int nchains, int N, int d) {
  const int nch = (N + 127) / 128;
  const size_t state = ((size_t)d * d + d) * sizeof(float);
  return (size_t)nchains * (self_segments(nchains, nch) + 1) * state;
}

cudaError_t launch_linear_self_tc(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d,
                                  int layout, int h_begin, int h_count, WsHeader* ws, size_t scratch_offset,
                                  cudaStream_t stream, const void* fq, const void* fk, int* first_grid) {
  if (first_grid) *first_grid = 0;
  if (h_count <= 0) return cudaSuccess;
  // fq, fk: feature tensors [B, h_count, N, d] that stand in for Q and K (feature map: identity)
  const bool features = fq != nullptr;
  CUtensorMap mq, mk, mv, mo;
  if (features ? (!make_feature_tensor_map(&mq, fq, B, H, N, d, h_begin, h_count, 128) ||
                  !make_feature_tensor_map(&mk, fk, B, H, N, d, h_begin, h_count, 128))
               : (!make_qkv_tensor_map(&mq, q, B, H, N, d, layout, 128) ||
                  !make_qkv_tensor_map(&mk, k, B, H, N, d, layout, 128)))
    return cudaErrorInvalidValue;
  if (!make_qkv_tensor_map(&mv, v, B, H, N, d, layout, 128) || !make_qkv_tensor_map(&mo, o, B, H, N, d, layout, 128))
    return cudaErrorInvalidValue;
  SelfParams p;
  p.N = N;
  p.nch = (N + 127) / 128;
  p.h_begin = h_begin;
  p.h_count = h_count;
  p.nchains = B * h_count;
  p.G = self_segments(p.nchains, p.nch);
  p.seg_base = p.nch / p.G;
  p.seg_rem = p.nch % p.G;
  p.nitems = p.nchains * p.G;
  const int state_floats = d * d + d;
  p.partial = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(ws) + scratch_offset);
  p.total = p.partial + (size_t)p.nitems * state_floats;
  p.status = &ws->status;
  int dev = 0, sms = 0;
  cudaError_t e;
  if ((e = device_info(&dev, &sms)) != cudaSuccess) return e;
  dim3 grid(p.nitems < sms ? p.nitems : sms);
  if (first_grid) *first_grid = (int)grid.x;
  auto launch_red = [&](auto kern, int smem, int threads) -> cudaError_t {
    cudaError_t err = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), dev, smem);
    if (err != cudaSuccess) return err;
    kern<<<grid, threads, smem, stream>>>(mk, mv, p);
    return cudaSuccess;
  };
  auto launch_out = [&](auto kern, int smem, int threads) -> cudaError_t {
    cudaError_t err = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), dev, smem);
    if (err != cudaSuccess) return err;
    kern<<<grid, threads, smem, stream>>>(mq, mo, p);
    return cudaSuccess;
  };
  if (features)
    e = (d == 64) ? launch_red(linear_self_reduce_kernel<64, true>, RedCfg<64>::kBytes, RedCfg<64>::kThreads)
                  : launch_red(linear_self_reduce_kernel<128, true>, RedCfg<128>::kBytes, RedCfg<128>::kThreads);
  else
    e = (d == 64) ? launch_red(linear_self_reduce_kernel<64, false>, RedCfg<64>::kBytes, RedCfg<64>::kThreads)
                  : launch_red(linear_self_reduce_kernel<128, false>, RedCfg<128>::kBytes, RedCfg<128>::kThreads);
  if (e != cudaSuccess) return e;
  note_launch();
  linear_self_sum_kernel<<<dim3((state_floats / 4 + 255) / 256, p.nchains), 256, 0, stream>>>(p.partial, p.total, p.G,
                                                                                              state_floats);
  note_launch();
  if (features)
    e = (d == 64) ? launch_out(linear_self_readout_kernel<64, true>, OutCfg<64>::kBytes, OutCfg<64>::kThreads)
                  : launch_out(linear_self_readout_kernel<128, true>, OutCfg<128>::kBytes, OutCfg<128>::kThreads);
  else
    e = (d == 64) ? launch_out(linear_self_readout_kernel<64, false>, OutCfg<64>::kBytes, OutCfg<64>::kThreads)
                  : launch_out(linear_self_readout_kernel<128, false>, OutCfg<128>::kBytes, OutCfg<128>::kThreads);
  if (e != cudaSuccess) return e;
  note_launch();
  return cudaGetLastError();
}

}  // namespace gf
