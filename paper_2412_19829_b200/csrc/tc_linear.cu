// Chunked causal linear attention on the tensor cores (bf16 in, fp32 accumulate and state).
//
// Algorithm 1 regrouped 128 rows at a time (exactly equal by associativity).  For chunk c with
// Qc = phi(Q_c), Kc = phi(K_c):
//   P   = Qc Kc^T                       (MMA1)   masked to j <= i           -> Pm (bf16)
//   S_c = S_{c-1} + Kc^T V_c            (MMA4)   fp32 master copy lives in TMEM for the whole chain
//   O   = Qc Sb_{c-1}  (+)  Pm V_c      (MMA2, MMA3)  Sb = bf16 copy of S in shared memory
//   den = rowsum(Pm) + Qc z_{c-1},  z_c = z_{c-1} + colsum(Kc)
//   out = O / den
// The denominators ride on the same tensor-core products as extra output columns (N = D + 16): V
// is followed by a constant box whose column 0 is all ones, so MMA4 leaves z = sum phi(K) in
// column D of the fp32 state and MMA3 adds rowsum(Pm) to column D of O; the bf16 copy of S is
// followed by a box holding z split in two bf16 terms (hi + lo: 16 bits), so MMA2 leaves Qc z in
// columns D, D + 1 of O.  The epilogue divides by the sum of those two columns.
// A (batch, head) chain is cut into segments of L chunks; a work item is one segment.  CTAs are
// persistent and take items round-robin in an order in which a segment's predecessor always has
// a smaller index, so the CTA that owns it is already running.  For an item the CTA
//   (A) applies phi to the segment's K tiles once, parks the results in the rows of the OUTPUT
//       tensor that this segment will later overwrite (no extra scratch, and the lines are still
//       in L2 when pass C reads them back) and accumulates the segment's own state contribution
//       dS | dz = sum Kc^T [V | 1] (not for a chain's last segment, whose contribution nobody needs),
//   (B) waits for the inclusive state of the previous segment in global scratch (one bounded
//       poller per CTA), publishes its own inclusive state = previous + dS and raises its flag,
//   (C) walks its chunks with the full pipeline starting from the previous segment's state,
//       reading phi(K) back instead of K, so every exponential of the layer is computed once.
// Warp roles:
//   warp 0       TMA producer (K, V tiles; rings of 2 K and 2 V slots at D = 128, 4 V slots at D = 64)
//   warp 1       MMA issuer
//   warps 2-5    "row group" (one thread per row): hands z over between segments, loads the state
//                before the segment; pass C: divides O by the denominator and stages it for the
//                store, one 64-column box at a time
//   warps 6-13   "Q group": pass C: requests the raw Q tiles and applies phi to them; the result goes
//                to TMEM as the A operand of MMA1/MMA2; pass A: transforms half of every K tile
//   warps 14-21  "K group": pass A: applies phi to the other half of every K tile (in place in
//                shared memory); pass C: masks/packs P in TMEM (two warps per TMEM lane quarter,
//                half of the key columns each), then converts the new S and z to bf16 for the next
//                chunk's readout
//   warp 22      TMA stores: parks phi(K) tiles (pass A), stores O boxes staged in the dead V
//                buffer (pass C)
//   warp 23      polls the previous segment's flag and raises this segment's flag
// TMEM (D=128): P 128 | O + denominators 144 | S + z 144 | phi(Q) 64 columns = 480.
// When the plan leaves every chain whole (kDirect): an item is a whole chain, there is no pass A,
// no parking and no hand-over; the phi warps transform each K tile in place one chunk ahead of
// the chunk pipeline (four K slots at D = 64).
// Every wait is bounded; on expiry the kernel records a status word and drains.
#include <mutex>

#include "common.cuh"
#include "sm100.cuh"

namespace gf {
namespace {

using namespace sm100;

constexpr int kThreads = 768;  // 24 warps, 80 registers each
constexpr int kMaxL = 32;      // most chunks per segment of a cut chain
constexpr float kLog2e = 1.4426950408889634f;
constexpr int kFlagStride = 32;  // one flag per 128-byte line

template <int D>
struct LinCfg {
  static constexpr int kTile = 128 * D * 2;  // one 128 x D bf16 tile
  static constexpr int kBoxBytes = 16384;    // one 128-row x 64-column box (what one TMA copy moves)
  static constexpr int kSbBox = D * 128;     // one D-row x 64-column box of Sb
  static constexpr int kSbBytes = D * D * 2;
  // The denominators ride along as 16 extra output columns (N = D + 16) of MMA2, MMA3 and MMA4,
  // whose B operands are rows of 64-column boxes a fixed distance (the descriptor's leading
  // byte offset) apart: V | ones and Sb | Zb.  The constant ones box (column 0 = 1) serves both
  // V slots, so it must lie one box distance past the last box of either: with B = kBoxBytes,
  //   D = 128:  V0a Q0 V1a V0b V1b Q1 ONES   (V0: distance 3B, V1: 2B; the Q boxes fill the holes)
  //   D = 64:   V0 V1 V2 V3 ONES             (slot s: distance (4 - s) B; a V tile is one box, and
  //                                           there is room for four slots)
  static constexpr int kVSlots = (D == 128) ? 2 : 4;
  __host__ __device__ static constexpr int v_off(int sv) { return (D == 128) ? (sv ? 2 : 0) * kBoxBytes : sv * kBoxBytes; }
  __host__ __device__ static constexpr int v_lbo(int sv) { return (D == 128) ? (sv ? 2 : 3) * kBoxBytes : (4 - sv) * kBoxBytes; }
  static constexpr int kOnes = (D == 128) ? 6 * kBoxBytes : 4 * kBoxBytes;
  static constexpr int kQ = (D == 128) ? kBoxBytes : 5 * kBoxBytes;  // raw Q landing buffer(s)
  static constexpr int kQStride = 4 * kBoxBytes;                     // between a tile's boxes (D = 128)
  static constexpr int kQLand = (D == 128) ? 1 : 2;                  // landing buffers (D = 64: one box each)
  // K ring of the chunk pipeline, contiguous: two stages; four in the one-pass form at D = 64, where there is
  // room and the pipeline runs at about one tile-load latency per chunk
  static constexpr int kKSlotsMax = (D == 128) ? 2 : 4;
  static constexpr int kK = (D == 128) ? 7 * kBoxBytes : 7 * kBoxBytes;
  static constexpr int kSb = kK + kKSlotsMax * kTile;  // bf16 copy of S, [D rows][D cols] in 64-column boxes
  static constexpr int kZb = kSb + kSbBytes;  // one more such box: column 0 = hi(z), column 1 = lo(z)
  // Pass A runs its K tiles through three slots: the two K slots and, third, the Sb buffer, which
  // is idle in that pass (at D = 64 Sb is smaller than a tile, so the third slot gets its own room)
  static constexpr int kKA2 = (D == 128) ? kSb : kZb + kSbBox;
  static constexpr int kBytes = ((D == 128) ? kZb + kSbBox : kKA2 + kTile) + 1024;
  // TMEM columns
  static constexpr int kQSlots = (D == 128) ? 1 : 2;  // phi(Q) operands in flight
  static constexpr int kNExt = D + 16;                // S and O with the denominator columns
  static constexpr uint32_t tP = 0, tO = 128, tS = 128 + kNExt, tQ = 128 + 2 * kNExt;  // tQ: kQSlots x D/2
  static constexpr uint32_t tOz = tO + D;  // [0] = Qc hi(z) + rowsum(Pm), [1] = Qc lo(z)
  static constexpr uint32_t tSz = tS + D;  // [0] = z (row = feature), the others stay zero
  static constexpr uint32_t kTmemCols = 512;
  // One published state: S then z.  S is stored [column/4][128 rows][4] so that the threads of a
  // warp (one row each, the TMEM lane order) touch consecutive 16-byte pieces.
  static constexpr int kStateZ = 128 * D;
  static constexpr int kStateFloats = 128 * D + D;
};

struct LinParams {
  int N, nch, h_begin, h_count, nchains;  // nchains: chains of this launch, the first being chain0 of the call
  int chain0;
  int G, nitems;         // segments per chain, nchains * G
  int seg_base, seg_rem; // the first seg_rem segments of a chain have seg_base + 1 chunks, the others seg_base
  float* S_io;           // [B, h_count, D, D] or null
  float* z_io;           // [B, h_count, D] or null
  int zero_init;
  unsigned int* status;  // two words: status, where
  unsigned int* flags;   // [nchains * G] x kFlagStride: 1 once the segment's inclusive state is in `prefix`
  float* prefix;         // [nchains * G][D*D + D]
};

struct LinItem {
  int g, chain, b, hl, h, c_begin, nC;
  bool last_seg, need_dS;
};


__device__ __forceinline__ LinItem decode_item(const LinParams& p, int item) {
  LinItem it;
  it.g = item / p.nchains;
  it.chain = item - it.g * p.nchains;
  const int call_chain = p.chain0 + it.chain;
  it.b = call_chain / p.h_count;
  it.hl = call_chain - it.b * p.h_count;
  it.h = p.h_begin + it.hl;
  it.c_begin = it.g * p.seg_base + (it.g < p.seg_rem ? it.g : p.seg_rem);
  it.nC = p.seg_base + (it.g < p.seg_rem ? 1 : 0);
  it.last_seg = (it.g == p.G - 1);
  it.need_dS = !it.last_seg;  // the last segment's contribution is needed by nobody
  return it;
}

struct LinBarriers {
  uint64_t q_full[2];  // raw Q tiles (landing buffer = chunk count % kQLand)
  uint64_t ka_full[5], kphi_full[5], ka_free[5];  // K tiles of pass A (slot = tile count % KA)
  uint64_t k_full[4], k_free[4];                  // K tiles of pass C (slot = chunk count % KS)
  uint64_t v_full[4], v_free[4];                  // V tiles of both passes (slot = tile count % kVSlots)
  uint64_t qphi_full[2], qphi_free[2];
  uint64_t p_full, s_full, o_full, mma2_done, a_done, pub_done, park_done, sb_idle, sb_parked;
  uint64_t pm_full, s_loaded, sb_full, s_final, o_free, o_staged[4][2];  // o_staged[V slot][box]
  uint64_t kd_phi[4];  // kDirect: a K tile of the chunk pipeline has been transformed in place
};

// Bounded poll of a monotonic counter in shared memory.
__device__ __forceinline__ bool wait_epoch_slow(const int* counter, int target, unsigned int* status,
                                                unsigned int where);
__device__ __forceinline__ bool wait_epoch(const int* counter, int target, unsigned int* status,
                                           unsigned int where) {
  if (*reinterpret_cast<const volatile int*>(counter) >= target) { __threadfence_block(); return true; }
  return wait_epoch_slow(counter, target, status, where);
}
__device__ __forceinline__ bool wait_epoch_slow(const int* counter, int target, unsigned int* status,
                                                unsigned int where) {
  const volatile int* c = counter;
  const long long t0 = clock64(), limit = wait_limit_cycles(status);
  while (*c < target) {
    if (clock64() - t0 > limit) {
      if (atomicCAS(status, 0u, 1u) == 0u) status[1] = where;
      return false;
    }
    __nanosleep(20);
  }
  __threadfence_block();
  return true;
}

// Bounded poll of a flag in global memory written by another CTA (acquire).
__device__ __forceinline__ bool wait_flag(const unsigned int* flag, unsigned int* status, unsigned int where) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
  if (v != 0u) return true;
  const long long t0 = clock64(), limit = wait_limit_cycles(status);
  while (true) {
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
    if (v != 0u) return true;
    if (clock64() - t0 > limit) {
      if (atomicCAS(status, 0u, 1u) == 0u) status[1] = where;
      return false;
    }
    __nanosleep(20);
  }
}


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

// kId: the tensors the kernel reads as Q and K already hold features (positive random features
// computed by a kernel of their own): the feature map here is the identity.
template <bool kId>
__device__ __forceinline__ uint32_t phi_sel(uint32_t w) {
  if constexpr (kId) return w;
  else return phi_bf16x2(w);
}

// phi on 64 rows (four groups of 16 from k8_begin on) x one 16-byte column chunk of a K tile, in
// place in shared memory (128B swizzle); rows past the end of the sequence become zero.
template <bool kId>
__device__ __forceinline__ void transform_k_rows(uint8_t* kb, int cin, int lane16, int k8_begin, int n_valid) {
  uint4 rawv[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int row = lane16 + 16 * (k8_begin + k);
    rawv[k] = *reinterpret_cast<const uint4*>(kb + row * 128 + ((cin ^ (row & 7)) << 4));
  }
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int row = lane16 + 16 * (k8_begin + k);
    const uint32_t keep = (row < n_valid) ? 0xffffffffu : 0u;
    rawv[k].x = phi_sel<kId>(rawv[k].x) & keep;
    rawv[k].y = phi_sel<kId>(rawv[k].y) & keep;
    rawv[k].z = phi_sel<kId>(rawv[k].z) & keep;
    rawv[k].w = phi_sel<kId>(rawv[k].w) & keep;
  }
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int row = lane16 + 16 * (k8_begin + k);
    *reinterpret_cast<uint4*>(kb + row * 128 + ((cin ^ (row & 7)) << 4)) = rawv[k];
  }
  fence_proxy_async_smem();
}

// Critical path of the segment hand-over, run by the 16 phi warps (4 per TMEM lane quarter, each
// thread one row x 32 columns): inclusive state of this segment = inclusive state of the previous
// one (global scratch, or the caller's initial state for the first segment) + this segment's own
// contribution (still in TMEM after pass A).  One batch of loads, one batch of stores, a fence and
// an arrival; the flag itself is raised by the store warp once every warp has arrived.
template <int D>
__device__ __forceinline__ bool publish_inclusive(const LinParams& p, const LinItem& it, LinBarriers& bar,
                                                  uint32_t tmem, int warp, int lane, uint32_t a_parity,
                                                  const int* prev_epoch, int item_number) {
  using C = LinCfg<D>;
  const int quarter = warp & 3, colq = (warp - 6) >> 2;  // colq 0..3: which 32 columns (D=128) / 16 (D=64)
  const int r = quarter * 32 + lane;
  constexpr int W = D / 4;  // columns per thread
  const long long slot = (long long)it.chain * p.G + it.g;
  bool ok = mbar_wait(&bar.a_done, a_parity, p.status, 600);
  tc_fence_after_sync();
  // one thread of the CTA (flag warp) polls the previous segment's flag for everybody
  ok = ok && wait_epoch(prev_epoch, item_number + 1, p.status, 601);
  if (ok) {
    uint32_t ds[W];
    if constexpr (D == 128) {
      uint32_t(&d32)[32] = *reinterpret_cast<uint32_t(*)[32]>(ds);
      tmem_ld32(tmem + C::tS + ((uint32_t)(quarter * 32) << 16) + colq * 32, d32);
    } else {
      tmem_ld16(tmem + C::tS + ((uint32_t)(quarter * 32) << 16) + colq * 16, ds);
    }
    if (r < D) {
      const float* Sin = nullptr;
      long long sin_stride = 1;  // in float4 units between consecutive column groups of one row
      if (it.g > 0) {
        Sin = p.prefix + (slot - 1) * C::kStateFloats + ((long long)(colq * (W / 4)) * 128 + r) * 4;
        sin_stride = 128;
      } else if (p.S_io != nullptr && !p.zero_init) {
        Sin = p.S_io + (((long long)it.b * p.h_count + it.hl) * D + r) * D + colq * W;  // caller's row-major state
      }
      float4 in[W / 4];
#pragma unroll
      for (int j = 0; j < W / 4; ++j)
        in[j] = (Sin != nullptr) ? __ldcg(reinterpret_cast<const float4*>(Sin) + j * sin_stride)
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
      tmem_wait_ld();
      float* Sout = p.prefix + slot * C::kStateFloats + ((long long)(colq * (W / 4)) * 128 + r) * 4;
#pragma unroll
      for (int j = 0; j < W / 4; ++j)
        __stcg(reinterpret_cast<float4*>(Sout) + j * 128,
               make_float4(in[j].x + __uint_as_float(ds[4 * j]), in[j].y + __uint_as_float(ds[4 * j + 1]),
                           in[j].z + __uint_as_float(ds[4 * j + 2]), in[j].w + __uint_as_float(ds[4 * j + 3])));
    } else {
      tmem_wait_ld();
    }
    // No per-thread gpu-scope fence here (hundreds of sequentially consistent fences at once cost
    // microseconds): the arrival below releases these stores at CTA scope to the store warp, whose
    // single st.release.gpu on the flag then publishes them (release is cumulative).
    tc_fence_before_sync();
  }
  __syncwarp();
  if (ok && lane == 0) mbar_arrive(&bar.pub_done);
  return ok;
}

template <int D, bool kDirect, bool kId>
__global__ void __launch_bounds__(kThreads, 1)
linear_tc_kernel(const __grid_constant__ CUtensorMap mq, const __grid_constant__ CUtensorMap mk,
                 const __grid_constant__ CUtensorMap mv, const __grid_constant__ CUtensorMap mo,
                 const LinParams p) {
  using C = LinCfg<D>;
  extern __shared__ uint8_t raw_smem[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(raw_smem) + 1023) & ~(uintptr_t)1023);
  uint8_t* sK = sm + C::kK;
  // box x of V slot sv (also the staging buffer of the O tile), of the Q landing buffer
  auto v_box = [&](int sv, int x) -> uint8_t* { return sm + C::v_off(sv) + x * C::v_lbo(sv); };
  constexpr int VS = C::kVSlots;
  constexpr int KS = (D == 64) ? 4 : 2;  // K ring of the chunk pipeline (its slots 0, 1 also serve pass A)
  auto q_box = [&](int slot, int x) -> uint8_t* { return sm + C::kQ + slot * C::kTile + x * C::kQStride; };
  constexpr int QL = C::kQLand;
  uint8_t* sSb = sm + C::kSb;
  __shared__ __align__(8) LinBarriers bar;
  uint8_t* sOnes = sm + C::kOnes;
  uint8_t* sZb = sm + C::kZb;
  __shared__ int prev_epoch;       // items whose predecessor state has been seen in global memory (monotonic)
  __shared__ int q_copied[2];      // per landing buffer: Q-group warps that have copied their part of a tile out (monotonic)
  __shared__ uint32_t tmem_base_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    atomicAdd(&p.status[5], 1u);  // WsHeader::placed: this CTA has an SM
    mbar_init(&bar.q_full[0], 1);
    mbar_init(&bar.q_full[1], 1);
    for (int s = 0; s < 5; ++s) {
      mbar_init(&bar.ka_full[s], 1);
      mbar_init(&bar.kphi_full[s], 16);
      mbar_init(&bar.ka_free[s], 2);  // the MMA issuer and the store warp
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bar.k_full[s], 1);
      mbar_init(&bar.v_full[s], 1);
      mbar_init(&bar.v_full[s + 2], 1);
      mbar_init(&bar.v_free[s + 2], 1);
      mbar_init(&bar.k_free[s], 1);
      mbar_init(&bar.v_free[s], 1);
      mbar_init(&bar.qphi_full[s], 8);
      mbar_init(&bar.qphi_free[s], 1);
    }
    mbar_init(&bar.sb_idle, 1);
    mbar_init(&bar.sb_parked, 1);
    for (int i = 0; i < 4; ++i) mbar_init(&bar.kd_phi[i], 16);
    for (int i = 2; i < 4; ++i) {
      mbar_init(&bar.k_full[i], 1);
      mbar_init(&bar.k_free[i], 1);
    }
    mbar_init(&bar.p_full, 1);
    mbar_init(&bar.s_full, 1);
    mbar_init(&bar.o_full, 1);
    mbar_init(&bar.mma2_done, 1);
    mbar_init(&bar.a_done, 1);
    mbar_init(&bar.pub_done, 20);  // 16 phi warps + 4 P-group warps
    mbar_init(&bar.park_done, 1);
    mbar_init(&bar.pm_full, 256);
    mbar_init(&bar.s_loaded, 256);
    mbar_init(&bar.sb_full, 256);
    mbar_init(&bar.s_final, 256);
    mbar_init(&bar.o_free, 128);
    for (int i = 0; i < 8; ++i) mbar_init(&bar.o_staged[i >> 1][i & 1], 128);
    prev_epoch = 0;
    q_copied[0] = q_copied[1] = 0;
    mbar_fence_init();
    tma_prefetch_desc(&mq);
    tma_prefetch_desc(&mk);
    tma_prefetch_desc(&mv);
    tma_prefetch_desc(&mo);
  }
  if (warp == 1) {
    tmem_alloc(&tmem_base_s, C::kTmemCols);
    tmem_relinquish();
  } else if (warp >= 2) {
    // constant ones box: column 0 of every key row is 1 (128B swizzle: the row's first 16-byte
    // chunk sits at position row & 7), all else 0; z operand cleared
    for (int i = tid - 64; i < C::kBoxBytes / 4; i += kThreads - 64) {
      const int row = i >> 5, w = i & 31;
      reinterpret_cast<uint32_t*>(sOnes)[i] = (w == ((row & 7) << 2)) ? 0x00003F80u : 0u;
    }
    for (int i = tid - 64; i < C::kSbBox / 4; i += kThreads - 64) reinterpret_cast<uint32_t*>(sZb)[i] = 0u;
    fence_proxy_async_smem();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_base_s;

  // Every role walks the same item list and keeps the same running counters: ta = K tiles of pass
  // A so far (slot = ta % KA, phase = ta / KA), nq = pass-C chunks so far (K slot = nq % KS, phase =
  // nq / KS), nv = V tiles of both passes so far (slot = nv % VS, phase = nv / VS).
  // pass A runs its K tiles through the K ring's slots and one more (KA in all)
  constexpr int KA = KS + 1;
  auto a_kslot = [&](uint32_t slot) -> uint8_t* { return slot < (uint32_t)KS ? sK + slot * C::kTile : sm + C::kKA2; };

  if (warp == 0) {
    // ================================================================ TMA producer
    if (elect_one()) {
      // A waiter may only use a parity wait on a barrier whose every phase it observes, so the K
      // tiles of the two passes complete (and are released) on barriers of their own.  A buffer that
      // serves both passes is only reloaded once its uses of either kind have drained: per barrier,
      // uses issued so far against phases already observed.
      uint32_t ta = 0, nv = 0, nq = 0, n_items = 0;
      uint32_t iss_a[5] = {0, 0, 0, 0, 0}, obs_a[5] = {0, 0, 0, 0, 0}, iss_c[4] = {0, 0, 0, 0}, obs_c[4] = {0, 0, 0, 0}, obs_sbi = 0;
      bool ok = true;
      auto drain = [&](uint64_t* b, uint32_t& obs, uint32_t issued, unsigned int where) -> bool {
        while (obs < issued) {
          if (!mbar_wait(b, obs & 1, p.status, where)) return false;
          ++obs;
        }
        return true;
      };
      // K, Q and the second read of V are streamed once; the first read of V (and the parked phi(K)
      // tiles) come back within the same item and should stay in L2 until then
      const uint64_t pol_stream = l2_policy_evict_first(), pol_keep = l2_policy_evict_last();
      for (int item = blockIdx.x; item < p.nitems && ok; item += gridDim.x) {
        const LinItem it = decode_item(p, item);
        for (int pass = kDirect ? 1 : 0; pass < 2 && ok; ++pass) {
          if (!kDirect && pass == 1 && !mbar_wait(&bar.park_done, n_items & 1, p.status, 103)) { ok = false; break; }
          for (int j = 0; j < it.nC; ++j) {
            const int n0 = (it.c_begin + j) * 128;
            if (pass == 0) {
              const uint32_t sa = ta % KA;
              // the slot's earlier pass-A uses, and what shares the buffer in pass C: a K slot, or
              // (third slot) the Sb operand, idle once the previous item's last readout is done
              // (sb_idle completes once per item whether or not the item's tiles reach this slot, so
              // several of its phases may be outstanding: they complete in order, only the last one
              // is waited for -- a parity wait on an older phase could block on the current one)
              ok = drain(&bar.ka_free[sa], obs_a[sa], iss_a[sa], 101);
              if (ok && sa < KS) ok = drain(&bar.k_free[sa], obs_c[sa], iss_c[sa], 104);
              if (ok && sa >= KS && obs_sbi < n_items) {
                ok = mbar_wait(&bar.sb_idle, (n_items - 1) & 1, p.status, 105);
                obs_sbi = n_items;
              }
              if (!ok) break;
              mbar_arrive_expect_tx(&bar.ka_full[sa], C::kTile);
              for (int x = 0; x < D / 64; ++x)
                tma_load_4d_hint(a_kslot(sa) + x * C::kBoxBytes, &mk, &bar.ka_full[sa], x * 64, n0, it.h, it.b,
                                 pol_stream);
              ++iss_a[sa];
              ++ta;
            } else {
              const uint32_t sc = nq % KS;
              ok = drain(&bar.k_free[sc], obs_c[sc], iss_c[sc], 104) &&
                   (kDirect || drain(&bar.ka_free[sc], obs_a[sc], iss_a[sc], 101));
              if (!ok) break;
              mbar_arrive_expect_tx(&bar.k_full[sc], C::kTile);
              for (int x = 0; x < D / 64; ++x)  // the phi(K) tile parked in the output rows (kDirect: raw K)
                tma_load_4d_hint(sK + sc * C::kTile + x * C::kBoxBytes, kDirect ? &mk : &mo, &bar.k_full[sc], x * 64, n0,
                                 it.h, it.b, pol_stream);
              ++iss_c[sc];
              ++nq;
            }
            if (pass == 1 || it.need_dS) {
              const int sv = nv % VS;
              if (nv >= VS && !mbar_wait(&bar.v_free[sv], ((nv / VS) + 1) & 1, p.status, 102)) { ok = false; break; }
              mbar_arrive_expect_tx(&bar.v_full[sv], C::kTile);
              for (int x = 0; x < D / 64; ++x)
                tma_load_4d_hint(v_box(sv, x), &mv, &bar.v_full[sv], x * 64, n0, it.h, it.b,
                                 pass == 0 ? pol_keep : pol_stream);
              ++nv;
            }
          }
        }
        ++n_items;
      }
    }
  } else if (warp == 1) {
    // ================================================================ MMA issuer
    if (elect_one()) {
      constexpr uint32_t id_p = umma_idesc_bf16(128, 128, false, false);  // P  = Qc Kc^T
      constexpr uint32_t id_s = umma_idesc_bf16(128, C::kNExt, true, true);   // [S | z] += Kc^T [V | 1]
      constexpr uint32_t id_o = umma_idesc_bf16(128, C::kNExt, false, true);  // [O | den] = Qc [Sb | Zb], += Pm [V | 1]
      constexpr uint32_t kLboA = (D == 128) ? C::kBoxBytes : 0;           // D=64: rows 64..127 of S mirror 0..63
      constexpr int QS = C::kQSlots;
      uint32_t ta = 0, nv = 0, nq = 0, n_sl = 0, n_sb = 0, n_of = 0, n_pm = 0;
      bool ok = true, first_item = true;
      [[maybe_unused]] uint32_t n_items = 0;
      for (int item = blockIdx.x; item < p.nitems && ok; item += gridDim.x, ++n_items) {
        const LinItem it = decode_item(p, item);
        if (!first_item) {
          // the previous item's last S conversion has read TMEM and written Sb: consume its phases
          ok = mbar_wait(&bar.s_loaded, n_sl & 1, p.status, 210) && mbar_wait(&bar.sb_full, n_sb & 1, p.status, 211);
          ++n_sl;
          ++n_sb;
          if (!ok) break;
        }
        first_item = false;
        // ---- pass A: dS = sum Kc^T V over the segment, from zero (only if somebody needs it)
        for (int j = 0; j < (kDirect ? 0 : it.nC); ++j) {
          const uint32_t sa = ta % KA;
          if (!mbar_wait(&bar.kphi_full[sa], (ta / KA) & 1, p.status, 220)) { ok = false; break; }
          if (it.need_dS) {
            const int sv = nv % VS;
            const uint32_t kbase = smem_u32(a_kslot(sa)), vbase = smem_u32(v_box(sv, 0));
            const uint32_t vlbo = C::v_lbo(sv);
            if (!mbar_wait(&bar.v_full[sv], (nv / VS) & 1, p.status, 221)) { ok = false; break; }
            tc_fence_after_sync();
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
              umma_ss(tmem + C::tS, umma_smem_desc(kbase + ks * 2048, kLboA, 1024),
                      umma_smem_desc(vbase + ks * 2048, vlbo, 1024), id_s, (j > 0) || (ks > 0));
            umma_commit(&bar.ka_free[sa]);  // second arrival: the store warp, once the tile is parked
            umma_commit(&bar.v_free[sv]);
            ++nv;
          } else {
            mbar_arrive(&bar.ka_free[sa]);
          }
          ++ta;
        }
        if (!ok) break;
        if (it.need_dS) umma_commit(&bar.a_done);
        // ---- pass C
        for (int j = 0; j < it.nC; ++j) {
          const int sv = nv % VS, sk = nq % KS, sq = nq % QS;  // slots of the V ring, of this pass's K ring, of phi(Q)
          const uint32_t kbase = smem_u32(sK) + sk * C::kTile, vbase = smem_u32(v_box(sv, 0));
          const uint32_t vlbo = C::v_lbo(sv);
          const uint32_t tq = tmem + C::tQ + sq * (D / 2);
          // the chunk's phi(K) tile: read back from the park, or (kDirect) transformed in place
          if (!mbar_wait(&bar.qphi_full[sq], (nq / QS) & 1, p.status, 200) ||
              !mbar_wait(kDirect ? &bar.kd_phi[sk] : &bar.k_full[sk], (nq / KS) & 1, p.status, 201)) {
            ok = false;
            break;
          }
          tc_fence_after_sync();
#pragma unroll 2
          for (int ks = 0; ks < D / 16; ++ks)
            umma_ts(tmem + C::tP, tq + ks * 8,
                    umma_smem_desc(kbase + (ks >> 2) * C::kBoxBytes + (ks & 3) * 32, 16, 1024), id_p, ks > 0);
          umma_commit(&bar.p_full);
          if (!mbar_wait(&bar.v_full[sv], (nv / VS) & 1, p.status, 202) ||
              !mbar_wait(&bar.s_loaded, n_sl & 1, p.status, 203)) {
            ok = false;
            break;
          }
          ++n_sl;
          tc_fence_after_sync();
#pragma unroll 2
          for (int ks = 0; ks < 8; ++ks)
            umma_ss(tmem + C::tS, umma_smem_desc(kbase + ks * 2048, kLboA, 1024),
                    umma_smem_desc(vbase + ks * 2048, vlbo, 1024), id_s, true);
          umma_commit(&bar.s_full);
          umma_commit(&bar.k_free[sk]);
          if (!mbar_wait(&bar.sb_full, n_sb & 1, p.status, 204)) { ok = false; break; }
          ++n_sb;
          if (nq >= 1) {
            if (!mbar_wait(&bar.o_free, n_of & 1, p.status, 205)) { ok = false; break; }
            ++n_of;
          }
          tc_fence_after_sync();
#pragma unroll 2
          for (int ks = 0; ks < D / 16; ++ks)
            umma_ts(tmem + C::tO, tq + ks * 8, umma_smem_desc(smem_u32(sSb) + ks * 2048, C::kSbBox, 1024), id_o,
                    ks > 0);
          umma_commit(&bar.mma2_done);
          umma_commit(&bar.qphi_free[sq]);
          if (j == it.nC - 1) umma_commit(&bar.sb_idle);  // Sb may now take a K tile of the next pass A
          if (!mbar_wait(&bar.pm_full, n_pm & 1, p.status, 206)) { ok = false; break; }
          ++n_pm;
          tc_fence_after_sync();
#pragma unroll 2
          for (int ks = 0; ks < 8; ++ks)
            umma_ts(tmem + C::tO, tmem + C::tP + (ks >> 2) * 64 + (ks & 3) * 8,
                    umma_smem_desc(vbase + ks * 2048, vlbo, 1024),
                    id_o, true);
          umma_commit(&bar.o_full);
          ++nv;
          ++nq;
        }
      }
    }
  } else if (warp < 6) {
    // ================================================================ row group (one thread per row)
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const bool s_row = r < D;  // rows of S are feature indices a < D
    // this feature's row of the z operand: columns 0 and 1 = hi(z), lo(z) (16 bits between them)
    uint32_t* zb_word = reinterpret_cast<uint32_t*>(sZb + swz128_offset(r, 0));
    auto put_z = [&](float z) {
      const float hi = __bfloat162float(__float2bfloat16_rn(z));
      *zb_word = pack_bf16(hi, z - hi);
    };
    uint32_t nv = 0, nq = 0, n_a = 0, n_items = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < p.nitems; item += gridDim.x) {
      const LinItem it = decode_item(p, item);
      const long long sidx = (long long)it.b * p.h_count + it.hl;
      const long long slot = (long long)it.chain * p.G + it.g;
      // ---- hand-over of z (column 0 of tSz, one feature per thread): this segment's own sum is
      //      there after pass A; previous segment's inclusive z in, this segment's inclusive z out
      if (it.need_dS) ok = mbar_wait(&bar.a_done, n_a & 1, p.status, 311);
      ok = ok && wait_epoch(&prev_epoch, (int)n_items + 1, p.status, 312);
      if (named_bar_or(1, 128, !ok)) break;
      float z0 = 0.f;
      if (s_row) {
        if (it.g > 0) z0 = __ldcg(p.prefix + (slot - 1) * C::kStateFloats + C::kStateZ + r);
        else if (p.z_io != nullptr && !p.zero_init) z0 = p.z_io[sidx * D + r];
      }
      if (it.need_dS) {
        tc_fence_after_sync();
        const float dz = __uint_as_float(tmem_ld1(tmem + C::tSz + lane_off));
        tmem_wait_ld();
        if (s_row) __stcg(p.prefix + slot * C::kStateFloats + C::kStateZ + r, z0 + dz);
        __syncwarp();
        if (lane == 0) mbar_arrive(&bar.pub_done);
      }
      // ---- hand-over of S: the 16 phi warps publish the inclusive state (they read dS from TMEM:
      //      do not overwrite it before they are done); this group loads the state before the segment
      if (it.need_dS) {
        ok = mbar_wait(&bar.pub_done, n_a & 1, p.status, 313);
        ++n_a;
        tc_fence_after_sync();
        nv += it.nC;
      }
      // Sb held K tiles in pass A: they have been parked (and, above, consumed by the tensor core)
      if (!kDirect) ok = mbar_wait(&bar.sb_parked, n_items & 1, p.status, 314) && ok;
      // the K group has read the previous item's last state out of TMEM
      if (n_items > 0) ok = mbar_wait(&bar.s_final, (n_items - 1) & 1, p.status, 315) && ok;
      tc_fence_after_sync();
      {
        const float* Sin = nullptr;
        long long sin_stride = 1;  // float4 units between consecutive column groups of one row
        if (it.g > 0) {
          Sin = p.prefix + (slot - 1) * C::kStateFloats + (long long)r * 4;
          sin_stride = 128;
        } else if (p.S_io != nullptr && !p.zero_init) {
          Sin = p.S_io + (sidx * D + r) * D;  // caller's row-major state
        }
#pragma unroll(D == 128 ? 1 : 2)
        for (int cc = 0; cc < D / 32; ++cc) {
          uint32_t v[32];
#pragma unroll
          for (int jj = 0; jj < 32; jj += 4) {
            float4 in = make_float4(0.f, 0.f, 0.f, 0.f);
            if (Sin != nullptr && s_row)
              in = __ldcg(reinterpret_cast<const float4*>(Sin) + (cc * 8 + jj / 4) * sin_stride);
            v[jj] = __float_as_uint(in.x);
            v[jj + 1] = __float_as_uint(in.y);
            v[jj + 2] = __float_as_uint(in.z);
            v[jj + 3] = __float_as_uint(in.w);
          }
          tmem_st32(tmem + C::tS + lane_off + cc * 32, v);
          if (cc == 0) {
            uint32_t zc[16];
#pragma unroll
            for (int jj = 1; jj < 16; ++jj) zc[jj] = 0u;
            zc[0] = __float_as_uint(z0);
            tmem_st16(tmem + C::tSz + lane_off, zc);
            if (s_row) put_z(z0);
          }
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
          }
        }
        tmem_wait_st();
        fence_proxy_async_smem();
        tc_fence_before_sync();
        mbar_arrive_cnt(&bar.s_loaded, 2);  // these barriers count the K group's 256 threads
        mbar_arrive_cnt(&bar.sb_full, 2);
      }
      // ---- pass C
      for (int j = 0; j < it.nC; ++j) {
        const int sv = nv % VS;
        // ---- O: divide by the denominator, bf16, stage for the TMA store
        if (!mbar_wait(&bar.o_full, nq & 1, p.status, 304)) {
          ok = false;
          break;
        }
        tc_fence_after_sync();
        uint32_t den_hi, den_lo;
        tmem_ld2(tmem + C::tOz + lane_off, den_hi, den_lo);
        tmem_wait_ld();
        const float inv = 1.f / (__uint_as_float(den_hi) + __uint_as_float(den_lo));
#pragma unroll 1
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
            *reinterpret_cast<uint4*>(v_box(sv, cc >> 1) + swz128_offset(r, (cc & 1) * 32 + g * 8)) = val;
          }
          if (cc == D / 32 - 1) {
            tc_fence_before_sync();
            mbar_arrive(&bar.o_free);
          }
          if (cc & 1) {
            fence_proxy_async_smem();
            mbar_arrive(&bar.o_staged[sv][cc >> 1]);
          }
        }
        ++nv;
        ++nq;
      }
      if (!ok) break;
      ++n_items;
    }
  } else if (warp < 22) {
    // ================================================================ phi warps: Q group (warps 6-13), K group (14-21)
    // Pass A and the hand-over of S are common to the two groups (one copy of the code); in pass
    // C the Q group applies phi to Q and the K group masks P.
    const bool kgrp = warp >= 14;
    const int tt = kgrp ? tid - 14 * 32 : tid - 6 * 32;  // 0..255 within the group
    const int quarter = warp & 3;                        // TMEM lane quarter of this warp
    const int half = ((warp - 6) >> 2) & 1;  // Q group: half of the head dimension; K group: half of the key columns
    const int colh = half;
    const int r = quarter * 32 + lane;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    constexpr int kChunksPerHalf = D / 16;  // 16-byte chunks of one row handled per Q-group thread
    uint32_t nq = 0, ta = 0, n_a = 0, n_items = 0;
    bool ok = true;
    // Raw Q tiles are requested by the Q group itself: the first QL tiles of this CTA's work here,
    // every later one by the warp that frees a landing buffer.  `step` moves (item, chunk of the
    // item) to the CTA's next chunk; false when there is none.
    auto step = [&](int& w_item, int& w_j, LinItem& w_it) -> bool {
      if (++w_j < w_it.nC) return true;
      w_item += gridDim.x;
      if (w_item >= p.nitems) return false;
      w_it = decode_item(p, w_item);
      w_j = 0;
      return true;
    };
    auto request_q = [&](int slot, const LinItem& w_it, int w_j) {
      mbar_arrive_expect_tx(&bar.q_full[slot], C::kTile);
      for (int x = 0; x < D / 64; ++x)
        tma_load_4d_hint(q_box(slot, x), &mq, &bar.q_full[slot], x * 64, (w_it.c_begin + w_j) * 128, w_it.h, w_it.b,
                         l2_policy_evict_first());
    };
    if (tid == 6 * 32 && (int)blockIdx.x < p.nitems) {
      if constexpr (QL == 1) {
        const LinItem first = decode_item(p, blockIdx.x);
        mbar_arrive_expect_tx(&bar.q_full[0], C::kTile);
        for (int x = 0; x < D / 64; ++x)
          tma_load_4d_hint(q_box(0, x), &mq, &bar.q_full[0], x * 64, first.c_begin * 128, first.h, first.b,
                           l2_policy_evict_first());
      } else {
        int w_item = blockIdx.x, w_j = 0;
        LinItem w_it = decode_item(p, w_item);
        for (int slot = 0; slot < QL; ++slot) {
          request_q(slot, w_it, w_j);
          if (!step(w_item, w_j, w_it)) break;
        }
      }
    }
    for (int item = blockIdx.x; item < p.nitems && ok; item += gridDim.x) {
      const LinItem it = decode_item(p, item);
      // kDirect: phi on this group's half of the K tile with running index idx (chunk jrow of the
      // item) of the chunk pipeline, in place
      auto transform_direct = [&](uint32_t idx, int jrow) {
        const uint32_t sl = idx % KS;
        ok = ok && mbar_wait(&bar.k_full[sl], (idx / KS) & 1, p.status, 430);
        const int cc = tt >> 4;
        if (ok && tt < 2 * D)
          transform_k_rows<kId>(sK + sl * C::kTile + (cc >> 3) * C::kBoxBytes, cc & 7, tt & 15, kgrp ? 0 : 4,
                           p.N - (it.c_begin + jrow) * 128);
        __syncwarp();
        if (ok && lane == 0) mbar_arrive(&bar.kd_phi[sl]);
      };
      if (kDirect) transform_direct(nq, 0);
      // ---- pass A: the K group takes rows 0..63 (by sixteens) of every K tile, the Q group rows 64..127
      for (int j = 0; j < (kDirect ? 0 : it.nC); ++j) {
        const uint32_t sk = ta % KA;
        ok = ok && mbar_wait(&bar.ka_full[sk], (ta / KA) & 1, p.status, 410);
        const int cc = tt >> 4;  // logical 16-byte column chunk 0 .. D/8-1
        if (ok && tt < 2 * D)
          transform_k_rows<kId>(a_kslot(sk) + (cc >> 3) * C::kBoxBytes, cc & 7, tt & 15, kgrp ? 0 : 4,
                           p.N - (it.c_begin + j) * 128);
        __syncwarp();
        if (ok && lane == 0) mbar_arrive(&bar.kphi_full[sk]);  // the tile may go to the tensor core and be parked
        ++ta;
      }

      // ---- hand-over of S: the two groups publish the inclusive state (column quarters 0, 1 / 2, 3)
      if (it.need_dS) {
        ok = publish_inclusive<D>(p, it, bar, tmem, warp, lane, n_a & 1, &prev_epoch, (int)n_items);
        ++n_a;
      }
      if (kgrp) {
        ok = !__any_sync(0xffffffffu, !ok);
        if (!ok) break;
        // ---- pass C: causal mask inside the chunk, bf16 back into TMEM.
        //      This warp owns rows [32 q, 32 q + 32) x key columns [64 colh, 64 colh + 64).
        for (int j = 0; j < it.nC; ++j) {
          // kDirect: this group's half of the next chunk's K tile, while the tensor core forms P
          if (kDirect && j + 1 < it.nC) transform_direct(nq + 1, j + 1);
          if (!ok || !mbar_wait(&bar.p_full, nq & 1, p.status, 301)) { ok = false; break; }
          tc_fence_after_sync();
#pragma unroll 1
          for (int e = 0; e < 2; ++e) {
            // 32-column block cc: all kept left of the diagonal block, all dropped right of it,
            // triangular on it (warp-uniform choice)
            const int cc = 2 * colh + e;
            uint32_t pk[16];
            if (cc > quarter) {
  #pragma unroll
              for (int jj = 0; jj < 16; ++jj) pk[jj] = 0u;
            } else {
              uint32_t v[32];
              tmem_ld32(tmem + C::tP + lane_off + cc * 32, v);
              tmem_wait_ld();
              const bool diag = (cc == quarter);
  #pragma unroll
              for (int jj = 0; jj < 16; ++jj) {
                const float p0 = (!diag || 2 * jj <= lane) ? __uint_as_float(v[2 * jj]) : 0.f;
                const float p1 = (!diag || 2 * jj + 1 <= lane) ? __uint_as_float(v[2 * jj + 1]) : 0.f;
                pk[jj] = pack_bf16(p0, p1);
              }
            }
            // packed P stays inside this warp's own fp32 columns (keys 64h..64h+63 -> columns 64h..64h+31),
            // so the two warps of a lane quarter never touch each other's unread input
            tmem_st16(tmem + C::tP + lane_off + colh * 64 + e * 16, pk);
          }
          tmem_wait_st();
          tc_fence_before_sync();
          mbar_arrive(&bar.pm_full);
          // ---- S: the fp32 master stays in TMEM; once this chunk's readout has consumed the old
          //      bf16 copy, stream the new one (and z) into shared memory for the next chunk.
          //      This warp: rows [32 q, 32 q + 32) x columns [colh D/2, colh D/2 + D/2).
          if (!mbar_wait(&bar.s_full, nq & 1, p.status, 302) || !mbar_wait(&bar.mma2_done, nq & 1, p.status, 303)) {
            ok = false;
            break;
          }
          tc_fence_after_sync();
          {
            // after the item's last chunk nobody reads Sb again (it may already hold a K tile of the
            // next item's pass A), and only a chain's last segment still wants the state itself
            const bool s_row = r < D;  // rows of S are feature indices a < D
            const long long sidx = (long long)it.b * p.h_count + it.hl;
            const bool last_chunk = (j == it.nC - 1);
            const bool write_final = it.last_seg && last_chunk && p.S_io != nullptr;
            if (colh == 0 && (!last_chunk || (it.last_seg && p.z_io != nullptr))) {
              const float z = __uint_as_float(tmem_ld1(tmem + C::tSz + lane_off));
              tmem_wait_ld();
              if (s_row) {
                if (!last_chunk) {
                  const float hi = __bfloat162float(__float2bfloat16_rn(z));  // columns 0, 1 = hi(z), lo(z)
                  *reinterpret_cast<uint32_t*>(sZb + swz128_offset(r, 0)) = pack_bf16(hi, z - hi);
                } else {
                  p.z_io[sidx * D + r] = z;
                }
              }
            }
#pragma unroll 1
            for (int e = 0; e < D / 64; ++e) {
              if (last_chunk && !write_final) break;
              const int cc = colh * (D / 64) + e;  // 32-column block
              uint32_t v[32];
              tmem_ld32(tmem + C::tS + lane_off + cc * 32, v);
              tmem_wait_ld();
              if (s_row && !last_chunk) {
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                  uint4 val;
                  val.x = pack_bf16(__uint_as_float(v[8 * g + 0]), __uint_as_float(v[8 * g + 1]));
                  val.y = pack_bf16(__uint_as_float(v[8 * g + 2]), __uint_as_float(v[8 * g + 3]));
                  val.z = pack_bf16(__uint_as_float(v[8 * g + 4]), __uint_as_float(v[8 * g + 5]));
                  val.w = pack_bf16(__uint_as_float(v[8 * g + 6]), __uint_as_float(v[8 * g + 7]));
                  *reinterpret_cast<uint4*>(sSb + (cc >> 1) * C::kSbBox + swz128_offset(r, (cc & 1) * 32 + g * 8)) = val;
                }
              }
              if (s_row && write_final) {
                float* dst = p.S_io + (sidx * D + r) * D + cc * 32;
#pragma unroll
                for (int jj = 0; jj < 32; jj += 4)
                  *reinterpret_cast<float4*>(dst + jj) =
                      make_float4(__uint_as_float(v[jj]), __uint_as_float(v[jj + 1]), __uint_as_float(v[jj + 2]),
                                  __uint_as_float(v[jj + 3]));
              }
            }
            tc_fence_before_sync();
            mbar_arrive(&bar.s_loaded);
            fence_proxy_async_smem();
            mbar_arrive(&bar.sb_full);
            if (last_chunk) mbar_arrive(&bar.s_final);
          }
          ++nq;
        }
        if (!ok) break;
      } else {
        ok = !__any_sync(0xffffffffu, !ok);
        if (!ok) break;
        for (int j = 0; j < it.nC && ok; ++j) {
          constexpr int QS = C::kQSlots;
          const int sq = nq % QS;
          const int ql = nq % QL;  // landing buffer of this chunk's tile
          ok = mbar_wait(&bar.q_full[ql], (nq / QL) & 1, p.status, 400);
          if (ok) {
            // copy the raw row half out of the landing buffer; the last warp to have done so
            // starts the load of the tile that takes the buffer next (a later chunk's, or one of
            // this CTA's next item), so that it is in flight while this one is transformed
            uint32_t pk[kChunksPerHalf * 4];
#pragma unroll
            for (int g = 0; g < kChunksPerHalf; ++g) {
              const int gl = half * kChunksPerHalf + g;  // logical 16-byte chunk within the row (8 columns)
              const int box = gl >> 3, cin = gl & 7;
              const uint4 rawv =
                  *reinterpret_cast<const uint4*>(q_box(ql, box) + r * 128 + ((cin ^ (r & 7)) << 4));
              pk[g * 4 + 0] = rawv.x;
              pk[g * 4 + 1] = rawv.y;
              pk[g * 4 + 2] = rawv.z;
              pk[g * 4 + 3] = rawv.w;
            }
            __syncwarp();
            if (lane == 0) {
              __threadfence_block();
              const int before = atomicAdd(&q_copied[ql], 1);
              if constexpr (QL == 1) {
                if ((before & 7) == 7) {  // the buffer is free: next chunk's tile, or the next item's first
                  int n_item = item, n_chunk = it.c_begin + j + 1;
                  LinItem nx = it;
                  if (j + 1 == it.nC) {
                    n_item = item + gridDim.x;
                    if (n_item < p.nitems) {
                      nx = decode_item(p, n_item);
                      n_chunk = nx.c_begin;
                    }
                  }
                  if (n_item < p.nitems) {
                    __threadfence_block();
                    fence_proxy_async_smem();
                    mbar_arrive_expect_tx(&bar.q_full[0], C::kTile);
                    for (int x = 0; x < D / 64; ++x)
                      tma_load_4d_hint(q_box(0, x), &mq, &bar.q_full[0], x * 64, n_chunk * 128, nx.h, nx.b,
                                       l2_policy_evict_first());
                  }
                }
              } else if ((before & 7) == 7) {
                // the buffer is free: it takes the tile QL chunks ahead of this one
                int w_item = item, w_j = j;
                LinItem w_it = it;
                bool more = true;
                for (int a = 0; a < QL && more; ++a) more = step(w_item, w_j, w_it);
                if (more) {
                  __threadfence_block();
                  fence_proxy_async_smem();
                  request_q(ql, w_it, w_j);
                }
              }
            }
#pragma unroll
            for (int w = 0; w < kChunksPerHalf * 4; ++w) pk[w] = phi_sel<kId>(pk[w]);
            if (nq >= QS)  // MMA1/MMA2 of the slot's previous chunk are done with it
              ok = mbar_wait(&bar.qphi_free[sq], ((nq / QS) + 1) & 1, p.status, 401);
            tc_fence_after_sync();
            if (ok) {
              if constexpr (D == 128) {
                uint32_t(&pk32)[32] = *reinterpret_cast<uint32_t(*)[32]>(pk);
                tmem_st32(tmem + C::tQ + sq * (D / 2) + lane_off + half * 32, pk32);
              } else {
                tmem_st16(tmem + C::tQ + sq * (D / 2) + lane_off + half * 16, pk);
              }
              tmem_wait_st();
              tc_fence_before_sync();
              __syncwarp();
              if (lane == 0) mbar_arrive(&bar.qphi_full[sq]);
            }
          }
          if (kDirect && ok && j + 1 < it.nC) transform_direct(nq + 1, j + 1);
          ok = !__any_sync(0xffffffffu, !ok);
          ++nq;
        }
      }
      ++n_items;
    }
  } else if (warp == 22) {
    // ================================================================ TMA store warp
    if (elect_one()) {
      uint32_t ta = 0, nv = 0;
      [[maybe_unused]] uint32_t n_items = 0;
      uint32_t n_os[4] = {0, 0, 0, 0};
      bool ok = true;
      const uint64_t pol_keep = l2_policy_evict_last();  // parked phi(K) tiles are read back by pass C
      const uint64_t pol_out = l2_policy_evict_first();  // nobody reads O again: leave L2 to the tiles that come back
      for (int item = blockIdx.x; item < p.nitems && ok; item += gridDim.x) {
        const LinItem it = decode_item(p, item);
        // ---- pass A: park phi(K) tiles in the output rows of their chunk
        for (int j = 0; j < (kDirect ? 0 : it.nC); ++j) {
          const uint32_t sk = ta % KA;
          if (!mbar_wait(&bar.kphi_full[sk], (ta / KA) & 1, p.status, 520)) { ok = false; break; }
          for (int x = 0; x < D / 64; ++x)
            tma_store_4d_hint(&mo, a_kslot(sk) + x * C::kBoxBytes, x * 64, (it.c_begin + j) * 128, it.h, it.b,
                              pol_keep);
          tma_store_commit();
          tma_store_wait_read<0>();
          mbar_arrive(&bar.ka_free[sk]);
          ++ta;
        }
        if (!ok) break;
        tma_store_wait_all<0>();  // parked tiles are in memory before pass C asks for them
        mbar_arrive(&bar.park_done);
        mbar_arrive(&bar.sb_parked);  // ... and Sb, the third slot of the pass, has been read out
        if (it.need_dS) nv += it.nC;
        // ---- pass C: O tiles
        for (int j = 0; j < it.nC; ++j) {
          const int sv = nv % VS;
          for (int x = 0; x < D / 64 && ok; ++x) {
            ok = mbar_wait(&bar.o_staged[sv][x], n_os[sv] & 1, p.status, 500);
            if (ok) tma_store_4d_hint(&mo, v_box(sv, x), x * 64, (it.c_begin + j) * 128, it.h, it.b, pol_out);
          }
          if (!ok) break;
          ++n_os[sv];
          tma_store_commit();
          tma_store_wait_read<0>();
          mbar_arrive(&bar.v_free[sv]);  // the staging buffer may take the V tile two uses later
          ++nv;
        }
        ++n_items;
      }
      tma_store_wait_all<0>();
    }
  } else {
    // ================================================================ flag warp
    if (elect_one()) {
      uint32_t n_a = 0;
      int n_items = 0;
      for (int item = blockIdx.x; item < p.nitems; item += gridDim.x, ++n_items) {
        const LinItem it = decode_item(p, item);
        const long long slot = (long long)it.chain * p.G + it.g;
        // one poller per CTA: hundreds of threads spinning on a handful of L2 lines slow the whole chain
        if (it.g > 0 && !wait_flag(p.flags + (slot - 1) * kFlagStride, p.status, 511)) break;
        __threadfence_block();
        *reinterpret_cast<volatile int*>(&prev_epoch) = n_items + 1;
        if (it.need_dS) {
          // every warp of the hand-over has written its part of the inclusive state
          if (!mbar_wait(&bar.pub_done, n_a & 1, p.status, 510)) break;
          ++n_a;
          const unsigned int one = 1u;
          // (status[4]: failure injection for tests -- that segment's flag is never raised)
          if (reinterpret_cast<const volatile unsigned int*>(p.status)[4] != (unsigned int)slot + 1u)
            asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p.flags + slot * kFlagStride), "r"(one) : "memory");
        }
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, C::kTmemCols);
}

}  // namespace


bool tc_linear_supported(int N, int d, int dtype) {
  (void)N;
  return dtype == GF_BF16 && (d == 64 || d == 128);
}

// Segmentation of the chains: G segments per chain, their lengths differing by one chunk at most
// (the longest has *L_out chunks).  CTAs take items round-robin, so the kernel lasts about
// ceil(items / CTAs) rounds of one item each, an item costing its chunks plus the fixed cost h of a
// hand-over (about one chunk); but a chain is also a serial pipeline - first pass of a segment,
// one hand-over link per segment (about 0.65 chunk each), second pass - which bounds the time
// from below when there are few chains.  Among the segment counts allowed, take the one with the
// least max(rounds x (L + h) x spill, L + 0.65 G).  Segments are between 4 and 32 chunks long;
// spill > 1 charges segments too long for what the CTAs running at one time park (phi(K) and V of
// their segments) to stay in L2.  The plan must not depend on the device that is current when the workspace size is asked
// for, so without a CTA count it assumes the 148 SMs of a B200.
namespace {
constexpr int kPlanL8 = 8;  // segment length the scratch is sized for when chains are many
// cost of a chunk of an uncut chain, in two-pass chunks
constexpr double direct_chunk_cost(int d) { return d == 128 ? 0.8 : 0.83; }
// ... and in a round that only part of the CTAs take part in: at d = 128 a full round of uncut chains is bound by
// HBM (3.3 us per chunk on a B200), a thin one by the CTA's own pipeline (2.4 us); at d = 64 the CTA's pipeline
// bounds both
constexpr double direct_chunk_floor(int d) { return d == 128 ? 0.59 : 0.83; }
// fixed cost of an item (hand-over, pipeline refill) in chunks: a chunk is cheaper at d = 64, the hand-over hardly
constexpr double handover_cost(int d) { return d == 128 ? 1.1 : 1.6; }
// Range of segment counts the automatic plan chooses from.
void plan_range(int nchains, int nch, int* g_min_out, int* g_max_out) {
  const int g_min8 = (nch + kPlanL8 - 1) / kPlanL8;
  int g_max = (nch + 3) / 4;
  // long chains in numbers: stay within a quarter more segments than 8-chunk segments give (the
  // scratch grows with the segment count); few chains: as many segments as it takes to fill the GPU
  int cap = (5 * g_min8 + 3) / 4;
  const int fill = (296 + nchains - 1) / nchains;
  if (cap < fill) cap = fill;
  if (g_max > cap) g_max = cap;
  if (g_max < g_min8) g_max = g_min8;
  int g_min = (nch + kMaxL - 1) / kMaxL;
  if (g_min < 1) g_min = 1;
  *g_min_out = g_min;
  *g_max_out = g_max;
}
}  // namespace

namespace {
// Bytes of parked tiles that stay in L2 while a round of items runs: about 0.6 of the cache (80 MB of
// a B200's 126 MiB).  Asked of the current device once; the B200 figure when there is no device (the
// plan can be queried on a machine without one).
double l2_park_bytes() {
  static double cached = 0.0;  // (a benign race: every writer stores the same value)
  if (cached == 0.0) {
    int dev = 0, l2 = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev) == cudaSuccess &&
        l2 > 0)
      cached = 0.6056 * (double)l2;
    else
      cached = 80e6;
  }
  return cached;
}
// Best two-pass plan for nchains chains of nch chunks: its cost in two-pass chunks (1e300 and
// *G_out = 1 when the chains are too short to cut).
double best_cut(int nchains, int nch, int d, int kPlanSMs, int* G_out) {
    int g_min, g_max;
    plan_range(nchains, nch, &g_min, &g_max);
    int G = 1;
    double best = 1e300;
    for (int g = g_min > 2 ? g_min : 2; g <= g_max; ++g) {
      const long long items = (long long)nchains * g;
      const long long rounds = (items + kPlanSMs - 1) / kPlanSMs;
      const double L = (double)nch / g;
      // What the running CTAs park at one time should stay in L2 (l2_park_bytes): of a
      // longer segment the excess comes back from DRAM, up to 40 % more time per chunk when the
      // rounds bound the time (when the serial chain does, DRAM has slack and nothing is charged).
      const double l_cap = l2_park_bytes() / ((double)(items < kPlanSMs ? items : kPlanSMs) * 4.0 * 128.0 * d);
      const double spill = L > l_cap ? 1.0 + 0.4 * (1.0 - l_cap / L) : 1.0;
      const double by_rounds = (double)rounds * (L + handover_cost(d)) * spill, by_chain = L + 0.65 * g;
      const double cost = by_rounds > by_chain ? by_rounds : by_chain;
      if (cost < best * (1.0 - 1e-9)) {
        best = cost;
        G = g;
      }
    }
    *G_out = G;
    return best;
}

// Fixed cost, in two-pass chunks, of running the leftover chains as a launch of their own (the gap
// between the launches, the second kernel's start-up and its uneven end: about 15 us).
constexpr double kSecondLaunchCost = 6.0;
}  // namespace

// `*whole_out` leading chains are left whole (the one-pass form), the others are cut into *G_out
// segments (the two-pass form; *G_out = 1 and *whole_out = nchains when no chain is cut).
// An uncut chain needs neither the first pass nor a hand-over (the kernel transforms K inside the
// chunk pipeline): a chunk then costs direct_chunk_cost(d) of a two-pass one, so with many chains
// that is the cheaper plan even though a CTA then walks a whole chain.  With somewhat more chains
// than CTAs the full rounds go whole and only the leftover chains are cut, in a second launch.
void linear_tc_plan_parts(int nchains, int N, int d, int split, int ctas, int* whole_out, int* L_out, int* G_out,
                          bool shared) {
  const int nch = (N + 127) / 128;
  int G, whole = 0;
  if (split > 0) {
    const int L = split > kMaxL ? kMaxL : split;
    G = (nch + L - 1) / L;
  } else if (split < 0) {
    G = 1;  // never cut: the one-pass form whatever the shape
    whole = nchains;
  } else {
    const int kPlanSMs = ctas > 0 ? ctas : 148;
    double best = best_cut(nchains, nch, d, kPlanSMs, &G);
    const int full = nchains / kPlanSMs, rest = nchains % kPlanSMs;
    double last = 0.0;  // the round of the chains left over after the full rounds
    if (rest > 0) {
      last = direct_chunk_cost(d) * rest / kPlanSMs;
      if (last < direct_chunk_floor(d)) last = direct_chunk_floor(d);
    }
    const double full_cost = (double)nch * full * direct_chunk_cost(d);
    // With a round or more of chains and other kernels to fill the idle SMs of a thin last round, cutting every
    // chain only adds SM-time (measured in the hybrid layer at d = 64: 17-22 % slower than whole chains).
    // The same holds from half a round of chains on (measured at d = 64 with 78 to 104 chains: whole chains
    // 3-23 % faster than cut ones beside the windowed heads; with 65 chains the cut plan still wins).
    if (shared && (full > 0 || 2 * nchains >= kPlanSMs)) best = 1e300;
    if (full_cost + (double)nch * last <= best) {
      best = full_cost + (double)nch * last;
      G = 1;
      whole = nchains;
    }
    // When other kernels share the GPU (the windowed heads of the hybrid layer), their CTAs fill the SMs
    // that a thin last round of whole chains leaves idle, and cutting the leftover chains only pays when
    // they are few (measured with 3 of 16 heads windowed: a gain up to 13 % for 8 to 21 leftover
    // chains on 148 CTAs, a loss of 3 to 11 % from 34 on).
    if (full > 0 && rest > 0 && (!shared || 6 * rest <= kPlanSMs)) {
      int g_rest = 1;
      const double mixed = full_cost + kSecondLaunchCost + best_cut(rest, nch, d, kPlanSMs, &g_rest);
      if (g_rest > 1 && mixed < best) {
        G = g_rest;
        whole = full * kPlanSMs;
      }
    }
  }
  if (G < 1) G = 1;
  *whole_out = whole;
  *G_out = G;
  *L_out = (nch + G - 1) / G;
}

void linear_tc_plan(int nchains, int N, int d, int split, int ctas, int* L_out, int* G_out) {
  int whole;
  linear_tc_plan_parts(nchains, N, d, split, ctas, &whole, L_out, G_out, false);
}

namespace {
// Largest segment count the plan may pick for nchains chains (the scratch is laid out for it).
int plan_g_max(int nchains, int N, int split) {
  int L, G;
  linear_tc_plan(nchains, N, 128, split, 0, &L, &G);
  if (split <= 0) {
    int g_min;
    plan_range(nchains, (N + 127) / 128, &g_min, &G);
  }
  return G;
}

// Largest number of hand-over slots (chains x segments) a launch of a call on nchains chains may
// use, whatever the CTA count: all chains cut, or the r < nchains chains left over after the full
// rounds (plan_range gives those at most min(ceil(nch / 4), max(the cap for many chains,
// ceil(296 / r))) segments, and r x that stays below the bound taken here).
long long plan_slots_max(int nchains, int N, int split) {
  long long m = (long long)nchains * plan_g_max(nchains, N, split);
  if (split == 0 && nchains > 1) {
    const long long nch4 = ((N + 127) / 128 + 3) / 4, r = nchains - 1;
    const long long rest = r * nch4 < 296 + r ? r * nch4 : 296 + r;
    if (m < rest) m = rest;
  }
  return m;
}
}  // namespace

size_t linear_tc_flag_bytes(int nchains, int N, int split) {
  return (size_t)plan_slots_max(nchains, N, split) * kFlagStride * sizeof(unsigned int);
}

size_t linear_tc_workspace_bytes(int nchains, int N, int d, int split) {
  return linear_tc_flag_bytes(nchains, N, split) +
         (size_t)plan_slots_max(nchains, N, split) * ((size_t)128 * d + d) * sizeof(float);
}

namespace {
// The CTAs of a cut-chain launch wait for one another, so two such kernels must not share the SMs: each
// could hold some of them while its own unplaced CTAs wait for the rest.  Per device the launches are
// therefore chained by an event: a cut-chain kernel starts only when the previous one, from whatever
// stream or host thread, has finished.  (Not inside a stream capture, where an outside event cannot be
// waited for: there the order of the caller's graphs applies.)
struct CutChainOrder {
  std::mutex mu;
  cudaEvent_t last[64] = {};
};
CutChainOrder g_cut_order;
}  // namespace

cudaError_t launch_linear_tc(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d,
                             int layout, int h_begin, int h_count, float* S_io, float* z_io, bool zero_init,
                             int split, int max_ctas, WsHeader* ws, cudaStream_t stream, bool shared,
                             const void* fq, const void* fk, int* first_grid) {
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
  LinParams p;
  p.N = N;
  p.nch = (N + 127) / 128;
  p.h_begin = h_begin;
  p.h_count = h_count;
  const int nchains = B * h_count;
  int dev = 0, sms = 0;
  cudaError_t e;
  if ((e = device_info(&dev, &sms)) != cudaSuccess) return e;
  // One CTA per SM at most: every CTA must be resident for the segment hand-over to make progress.
  // (max_ctas > 0 leaves SMs to a kernel running beside this one.)
  if (max_ctas > 0 && max_ctas < sms) sms = max_ctas;
  int L_max = 0, whole = 0, G = 1;
  linear_tc_plan_parts(nchains, N, d, split, sms, &whole, &L_max, &G, shared);
  p.S_io = S_io;
  p.z_io = z_io;
  p.zero_init = zero_init ? 1 : 0;
  p.status = &ws->status;
  uint8_t* scratch = reinterpret_cast<uint8_t*>(ws) + sizeof(WsHeader);
  p.flags = reinterpret_cast<unsigned int*>(scratch);  // zeroed by the caller
  p.prefix = reinterpret_cast<float*>(scratch + linear_tc_flag_bytes(nchains, N, split));
  auto launch = [&](auto kern, size_t smem) -> cudaError_t {
    cudaError_t err = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), dev, (int)smem);
    if (err != cudaSuccess) return err;
    dim3 grid(p.nitems < sms ? p.nitems : sms);
    if (first_grid && *first_grid == 0) *first_grid = (int)grid.x;
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    if (p.G > 1 && (err = cudaStreamIsCapturing(stream, &capturing)) != cudaSuccess) return err;
    const bool chained = p.G > 1 && capturing == cudaStreamCaptureStatusNone;
    std::unique_lock<std::mutex> order;
    if (chained) {
      order = std::unique_lock<std::mutex>(g_cut_order.mu);
      cudaEvent_t& ev = g_cut_order.last[dev];
      if (ev == nullptr) {
        if ((err = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming)) != cudaSuccess) return err;
      } else if ((err = cudaStreamWaitEvent(stream, ev, 0)) != cudaSuccess) {
        return err;
      }
    }
    kern<<<grid, kThreads, smem, stream>>>(mq, mk, mv, mo, p);
    note_launch();
    err = cudaGetLastError();
    if (chained && err == cudaSuccess) err = cudaEventRecord(g_cut_order.last[dev], stream);
    return err;
  };
  // Chains [chain0, chain0 + count) of the call in one launch: whole (the one-pass form of the kernel) or cut
  // into g segments (the two-pass form).  The one-pass form neither reads nor writes the hand-over scratch.
  auto run = [&](int chain0, int count, int g, bool direct) -> cudaError_t {
    p.chain0 = chain0;
    p.nchains = count;
    p.G = g;
    p.seg_base = p.nch / g;
    p.seg_rem = p.nch % g;
    p.nitems = count * g;
    if (features) {
      if (d == 64)
        return direct ? launch(linear_tc_kernel<64, true, true>, LinCfg<64>::kBytes)
                      : launch(linear_tc_kernel<64, false, true>, LinCfg<64>::kBytes);
      return direct ? launch(linear_tc_kernel<128, true, true>, LinCfg<128>::kBytes)
                    : launch(linear_tc_kernel<128, false, true>, LinCfg<128>::kBytes);
    }
    if (d == 64)
      return direct ? launch(linear_tc_kernel<64, true, false>, LinCfg<64>::kBytes)
                    : launch(linear_tc_kernel<64, false, false>, LinCfg<64>::kBytes);
    return direct ? launch(linear_tc_kernel<128, true, false>, LinCfg<128>::kBytes)
                  : launch(linear_tc_kernel<128, false, false>, LinCfg<128>::kBytes);
  };
  // `whole` leading chains uncut (automatic plan only: a segment length asked for by the caller always takes
  // the two-pass form, also when it covers the whole chain), the others cut into G segments behind them
  if (whole > 0 && (e = run(0, whole, 1, true)) != cudaSuccess) return e;
  if (whole < nchains && (e = run(whole, nchains - whole, G, false)) != cudaSuccess) return e;
  return cudaSuccess;
}

}  // namespace gf
