// Windowed causal softmax attention on the tensor cores (bf16 in, fp32 accumulate).
//
// A work unit is one tile of 128 query rows of one (batch, head).  The keys a tile can see,
// [i0 - w + 1, i0 + 127], are walked in 128-key tiles aligned to the query grid:
//   S = Q K^T      tcgen05.mma, A and B from shared memory (K-major), S (128x128 fp32) in TMEM
//   P = softmax    two threads per query row (64 key columns each) read the S row from TMEM, mask
//                  (causal edge on the diagonal tile, window edge on the leftmost ones), agree on
//                  the row maximum through shared memory, exponentiate against a running
//                  reference maximum and write P as bf16 back over S in TMEM
//   O += P V       tcgen05.mma with A = P from TMEM, B = V from shared memory (MN-major)
// O stays in TMEM across key tiles; it is rescaled only when a row's maximum moves by more than
// 2^8 (lazy rescaling), which with bounded logits is rare.  Final rows are divided by the softmax
// denominator, packed to bf16, staged in the (by then dead) V buffer and written with a TMA store.
//
// CTAs are persistent: each draws query tiles from a global ticket counter until none are left,
// so that the fixed costs of a tile (TMEM allocation, the first loads, the output store) overlap
// the neighbouring tiles' work: Q and the first K tile of the next unit are loaded while the
// current one finishes, and the output store runs beside the next unit's first products.  CTAs
// never wait for one another, so any number of them may be resident at a time.
//
// Warp roles: warp 0 = TMA producer (also draws the tickets), warp 1 = MMA issuer, warps 2..9 =
// softmax/epilogue (two warps per TMEM lane quarter, one per half of the key columns / of the
// output columns).  TMEM use is 256 columns and shared memory under 113 KB so that two CTAs share
// an SM: while one is in its softmax the other owns the tensor core.
#include "common.cuh"
#include "sm100.cuh"

namespace gf {
namespace {

using namespace sm100;

constexpr int kThreads = 320;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleThreshold = 8.0f;  // log2 units
constexpr int kUnitRing = 4;               // no role is ever this many units behind the producer

__device__ __forceinline__ float ex2_approx(float x) {  // 2^x, flushes denormals, 2^-inf = 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Developer instrumentation (compiled only with -DGF_PROFILE): time stamps of the first key tiles
// of CTA 0, read back with gformer_debug_read_wprofile.
#ifdef GF_PROFILE
__device__ unsigned long long g_wprof[2][64][8];
__device__ __forceinline__ void wprof(int role, unsigned int kt, int ev) {
  if (blockIdx.x == 0 && kt < 64) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    g_wprof[role][kt][ev] = t;
  }
}
#define WPROF(role, kt, ev) wprof(role, kt, ev)
#else
#define WPROF(role, kt, ev)
#endif

template <int D>
struct WinSmem {
  static constexpr int kTile = 128 * D * 2;  // bytes of one 128 x D bf16 tile
  static constexpr int kQ = 0;
  static constexpr int kK = kTile;
  static constexpr int kV = 2 * kTile;
  static constexpr int kBytes = 3 * kTile + 1024;  // + alignment slack
};

struct WinParams {
  int N, w, tiles_back;  // tiles_back = number of key tiles before the diagonal one
  int fwd, tiles_fwd;    // keys after the query it may see (0: causal; w - 1: two-sided) and the tiles they span
  float scale_log2;
  int h_begin, h_count, nqt, total;  // work units: (batch, head, query tile), query tile fastest
  unsigned int* status;
  unsigned int* ticket;  // zero at launch; units beyond the first one of every CTA come from here
};

// Bounded poll of a monotonic counter in shared memory.
__device__ __forceinline__ bool win_wait_epoch(const int* counter, int target, unsigned int* status,
                                               unsigned int where) {
  const volatile int* c = counter;
  if (*c >= target) { __threadfence_block(); return true; }
  const long long t0 = clock64();
  while (*c < target) {
    if (clock64() - t0 > 4000000000LL) {
      if (atomicCAS(status, 0u, 1u) == 0u) status[1] = where;
      return false;
    }
    __nanosleep(20);
  }
  __threadfence_block();
  return true;
}

template <int D, bool kTwoSided>
__global__ void __launch_bounds__(kThreads, 2)
window_tc_kernel(const __grid_constant__ CUtensorMap mq, const __grid_constant__ CUtensorMap mk,
                 const __grid_constant__ CUtensorMap mv, const __grid_constant__ CUtensorMap mo,
                 const WinParams p) {
  extern __shared__ uint8_t raw_smem[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(raw_smem) + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = sm + WinSmem<D>::kQ;
  uint8_t* sK = sm + WinSmem<D>::kK;
  uint8_t* sV = sm + WinSmem<D>::kV;
  // per key tile: k_full, k_empty, v_full, v_empty, s_full, p_full, pv_done; per unit: q_full, q_empty,
  // o_full, o_free
  __shared__ __align__(8) uint64_t q_full, q_empty, k_full, k_empty, v_full, v_empty, s_full, p_full, pv_done, o_full,
      o_free;
  __shared__ uint32_t tmem_base_s;
  __shared__ float mx_s[2][2][128];  // [tile parity][column half][row]: half-row maxima
  __shared__ float l_s[2][128];      // [column half][row]: half-row sums at the end
  __shared__ int unit_ring[kUnitRing];  // the CTA's n-th work unit (-1: no more)
  __shared__ int units_posted;          // entries of unit_ring written so far (monotonic)

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    mbar_init(&q_full, 1);
    mbar_init(&q_empty, 1);
    mbar_init(&k_full, 1);
    mbar_init(&k_empty, 1);
    mbar_init(&v_full, 1);
    mbar_init(&v_empty, 1);
    mbar_init(&s_full, 1);
    mbar_init(&p_full, 256);
    mbar_init(&pv_done, 1);
    mbar_init(&o_full, 1);
    mbar_init(&o_free, 1);
    unit_ring[0] = blockIdx.x;  // the grid never exceeds the number of units
    units_posted = 1;
    mbar_fence_init();
    tma_prefetch_desc(&mq);
    tma_prefetch_desc(&mk);
    tma_prefetch_desc(&mv);
    tma_prefetch_desc(&mo);
  }
  if (warp == 1) {
    tmem_alloc(&tmem_base_s, 256);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_base_s;
  const uint32_t tS = tmem;        // 128 columns: S, later P (bf16 pairs)
  const uint32_t tO = tmem + 128;  // D columns

  // a unit's coordinates
  struct Unit {
    int qt, h, b, i0, t_first, n_tiles;
  };
  auto decode = [&](int u) {
    Unit x;
    x.qt = u % p.nqt;
    const int bh = u / p.nqt;
    x.h = p.h_begin + bh % p.h_count;
    x.b = bh / p.h_count;
    x.i0 = x.qt * 128;
    x.t_first = (x.qt - p.tiles_back) > 0 ? (x.qt - p.tiles_back) : 0;
    // kTwoSided: the tiles after the diagonal one that the window reaches, up to the sequence end
    const int t_last = !kTwoSided ? x.qt : ((x.qt + p.tiles_fwd) < p.nqt ? (x.qt + p.tiles_fwd) : p.nqt - 1);
    x.n_tiles = t_last - x.t_first + 1;
    return x;
  };
  auto unit_at = [&](uint32_t n) -> int {
    if (!win_wait_epoch(&units_posted, (int)n + 1, p.status, 90)) return -1;
    return reinterpret_cast<const volatile int*>(unit_ring)[n % kUnitRing];
  };

  // Every role walks the same list of units and keeps the same running counters: nu = units so
  // far, kt = key tiles so far (over all units).  All barriers are single-buffered: phase = count.
  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer + ticket drawer
    if (elect_one()) {
      const uint64_t pol_once = l2_policy_evict_first();  // Q is read once; K/V tiles by 5 query tiles
      uint32_t nu = 0, kt = 0;
      bool ok = true;
      for (int u = blockIdx.x; u >= 0 && ok;) {
        const Unit x = decode(u);
        // draw the next ticket now; its value is only needed once this unit's loads are out
        const unsigned int t_next = atomicAdd(p.ticket, 1u);
        if (nu >= 1 && !mbar_wait(&q_empty, (nu - 1) & 1, p.status, 12)) break;
        mbar_arrive_expect_tx(&q_full, WinSmem<D>::kTile);
        for (int c = 0; c < D / 64; ++c) tma_load_4d_hint(sQ + c * 16384, &mq, &q_full, c * 64, x.i0, x.h, x.b, pol_once);
        for (int it = 0; it < x.n_tiles; ++it, ++kt) {
          const int j0 = (x.t_first + it) * 128;
          if (kt >= 1 && !mbar_wait(&k_empty, (kt - 1) & 1, p.status, 10)) { ok = false; break; }
          mbar_arrive_expect_tx(&k_full, WinSmem<D>::kTile);
          for (int c = 0; c < D / 64; ++c) tma_load_4d(sK + c * 16384, &mk, &k_full, c * 64, j0, x.h, x.b);
          if (kt >= 1 && !mbar_wait(&v_empty, (kt - 1) & 1, p.status, 11)) { ok = false; break; }
          mbar_arrive_expect_tx(&v_full, WinSmem<D>::kTile);
          for (int c = 0; c < D / 64; ++c) tma_load_4d(sV + c * 16384, &mv, &v_full, c * 64, j0, x.h, x.b);
        }
        ++nu;
        u = (t_next < (unsigned int)(p.total - (int)gridDim.x)) ? (int)(gridDim.x + t_next) : -1;
        unit_ring[nu % kUnitRing] = ok ? u : -1;
        __threadfence_block();
        *reinterpret_cast<volatile int*>(&units_posted) = (int)nu + 1;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (elect_one()) {
      constexpr uint32_t idesc_qk = umma_idesc_bf16(128, 128, false, false);
      constexpr uint32_t idesc_pv = umma_idesc_bf16(128, D, false, true);
      uint32_t nu = 0, kt = 0;
      bool ok = true;
      for (; ok; ++nu) {
        const int u = unit_at(nu);
        if (u < 0) break;
        const Unit x = decode(u);
        if (!mbar_wait(&q_full, nu & 1, p.status, 20)) break;
        for (int it = 0; it < x.n_tiles; ++it, ++kt) {
          if (!mbar_wait(&k_full, kt & 1, p.status, 21)) { ok = false; break; }
          WPROF(0, kt, 0);
          tc_fence_after_sync();
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            const uint32_t off = (ks >> 2) * 16384 + (ks & 3) * 32;
            umma_ss(tS, umma_smem_desc(smem_u32(sQ) + off, 16, 1024), umma_smem_desc(smem_u32(sK) + off, 16, 1024),
                    idesc_qk, ks > 0);
          }
          umma_commit(&k_empty);
          umma_commit(&s_full);
          WPROF(0, kt, 1);
          if (it == x.n_tiles - 1) umma_commit(&q_empty);  // the next unit's Q may land
          if (!mbar_wait(&p_full, kt & 1, p.status, 22)) { ok = false; break; }
          WPROF(0, kt, 2);
          if (!mbar_wait(&v_full, kt & 1, p.status, 23)) { ok = false; break; }
          WPROF(0, kt, 3);
          // the first product of a unit overwrites O: the previous unit's epilogue has read it
          if (it == 0 && nu >= 1 && !mbar_wait(&o_free, (nu - 1) & 1, p.status, 24)) { ok = false; break; }
          tc_fence_after_sync();
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            umma_ts(tO, tS + (ks >> 2) * 64 + (ks & 3) * 8, umma_smem_desc(smem_u32(sV) + ks * 2048, 16384, 1024),
                    idesc_pv, (it > 0) || (ks > 0));
          }
          // the unit's last V buffer becomes the staging buffer of its output: the epilogue
          // releases it once the store has read it
          if (it < x.n_tiles - 1) umma_commit(&v_empty);
          umma_commit(&pv_done);
          WPROF(0, kt, 4);
          if (it == x.n_tiles - 1) umma_commit(&o_full);
        }
      }
    }
  } else {
    // ------------------------------------------------------------ softmax + epilogue
    const int quarter = warp & 3;    // TMEM lane quarter this warp may touch
    const int hh = (warp - 2) >> 2;  // half of the key columns (softmax) / of the output columns (epilogue)
    const int r = quarter * 32 + lane;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const int c0 = hh * 64, c1 = hh * 64 + 63;  // this thread's key columns within a tile
    uint32_t nu = 0, kt = 0;
    bool ok = true;
    for (; ok; ++nu) {
      const int u = unit_at(nu);
      if (u < 0) break;
      const Unit x = decode(u);
      const int i0 = x.i0, i = i0 + r;
      float m_ref = -INFINITY;  // reference maximum the stored O and l are relative to (same in both halves)
      float l = 0.f;            // sum over this thread's columns
      for (int it = 0; it < x.n_tiles; ++it, ++kt) {
        const int j0 = (x.t_first + it) * 128;
        if (!mbar_wait(&s_full, kt & 1, p.status, 30)) { ok = false; break; }
        if (tid == 64) WPROF(1, kt, 0);
        tc_fence_after_sync();
        // valid key columns of this row in this tile: [lo, hi]; over the warp's 32 rows lo and hi move
        // by 31, so the 64-column half is classified per warp: nothing visible (costs nothing), all
        // visible to every row (no per-element test), or mixed
        const int lo = i - p.w + 1 - j0;
        const int i_first = i0 + quarter * 32;  // the warp's first row
        // (two-sided window: the query also sees p.fwd keys after it, and keys past the end do not exist)
        const int hi = kTwoSided ? min(i + p.fwd, p.N - 1) - j0 : i - j0;
        const int lo_first = i_first - p.w + 1 - j0;  // lo of the warp's first row (last row: +31)
        const int hi_first = kTwoSided ? min(i_first + p.fwd, p.N - 1) - j0 : i_first - j0;  // hi of its first row
        const int hi_last = kTwoSided ? min(i_first + 31 + p.fwd, p.N - 1) - j0 : hi_first + 31;  // ... of its last row
        const bool none = (c1 < lo_first || c0 > hi_last);
        const bool inside = (c0 >= lo_first + 31) && (c1 <= hi_first);
        // Two sweeps over the half row (maximum, then exponentials): the scores stay in TMEM between
        // the sweeps, so that few registers are live across the exchange of the maxima.
        float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        if (!none) {
          uint32_t sa[32], sb[32];
          tmem_ld32(tS + lane_off + c0, sa);
          tmem_ld32(tS + lane_off + c0 + 32, sb);
          tmem_wait_ld();
          if (inside) {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              mx[j & 3] = fmaxf(mx[j & 3], __uint_as_float(sa[j]));
              mx[(j + 2) & 3] = fmaxf(mx[(j + 2) & 3], __uint_as_float(sb[j]));
            }
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const int col = c0 + j;
              if (col >= lo && col <= hi) mx[j & 3] = fmaxf(mx[j & 3], __uint_as_float(sa[j]));
              if (col + 32 >= lo && col + 32 <= hi) mx[(j + 2) & 3] = fmaxf(mx[(j + 2) & 3], __uint_as_float(sb[j]));
            }
          }
        }
        // the row maximum over both halves: exchange through shared memory with the partner warp
        // (same lane quarter, other half); double buffered by tile parity, one barrier per tile
        const float mloc = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
        mx_s[kt & 1][hh][r] = mloc;
        if (tid == 64) WPROF(1, kt, 1);
        asm volatile("bar.sync %0, 64;" ::"r"(2 + quarter) : "memory");
        if (tid == 64) WPROF(1, kt, 2);
        const float mt = fmaxf(mloc, mx_s[kt & 1][hh ^ 1][r]) * p.scale_log2;  // scale > 0
        // lazy rescale of what has been accumulated so far (both halves take the same decision)
        float alpha = 1.f;
        bool need = false;
        if (mt > m_ref + kRescaleThreshold) {  // also true for the first finite maximum
          need = (m_ref != -INFINITY);         // nothing accumulated yet otherwise (O row and l are 0)
          alpha = need ? exp2f(m_ref - mt) : 1.f;
          m_ref = mt;
          l *= alpha;
        }
        if (it > 0) {
          if (__any_sync(0xffffffffu, need)) {
            if (!mbar_wait(&pv_done, (kt - 1) & 1, p.status, 31)) { ok = false; break; }
            tc_fence_after_sync();
            // this warp's half of the output columns, a few at a time (rare path)
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
              uint32_t oreg[16];
              tmem_ld16(tO + lane_off + hh * (D / 2) + c * 16, oreg);
              tmem_wait_ld();
#pragma unroll
              for (int j = 0; j < 16; ++j) oreg[j] = __float_as_uint(__uint_as_float(oreg[j]) * alpha);
              tmem_st16(tO + lane_off + hh * (D / 2) + c * 16, oreg);
            }
            tmem_wait_st();
          }
        }
        // p = 2^(s * scale_log2 - m_ref), bf16, back over S: this thread's 64 scores become 32 packed
        // columns at [64 hh, 64 hh + 32), inside columns it has itself consumed
        const float neg_mref = (m_ref == -INFINITY) ? 0.f : -m_ref;
        float ls[4] = {0.f, 0.f, 0.f, 0.f};
        uint32_t sa[32], sb[32];
        if (!none) {
          tmem_ld32(tS + lane_off + c0, sa);
          tmem_ld32(tS + lane_off + c0 + 32, sb);
          tmem_wait_ld();
        }
        // packed in place: pair j of sa / sb goes to word j of the same array once it has been read
        if (none) {
#pragma unroll
          for (int j = 0; j < 16; ++j) sa[j] = sb[j] = 0u;
        } else if (inside) {  // the common case, kept free of any masking arithmetic
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float p0 = ex2_approx(fmaf(__uint_as_float(sa[2 * j]), p.scale_log2, neg_mref));
            const float p1 = ex2_approx(fmaf(__uint_as_float(sa[2 * j + 1]), p.scale_log2, neg_mref));
            const float p2 = ex2_approx(fmaf(__uint_as_float(sb[2 * j]), p.scale_log2, neg_mref));
            const float p3 = ex2_approx(fmaf(__uint_as_float(sb[2 * j + 1]), p.scale_log2, neg_mref));
            ls[j & 3] += (p0 + p1) + (p2 + p3);
            sa[j] = pack_bf16(p0, p1);
            sb[j] = pack_bf16(p2, p3);
          }
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            float a0 = fmaf(__uint_as_float(sa[2 * j]), p.scale_log2, neg_mref);
            float a1 = fmaf(__uint_as_float(sa[2 * j + 1]), p.scale_log2, neg_mref);
            float b0 = fmaf(__uint_as_float(sb[2 * j]), p.scale_log2, neg_mref);
            float b1 = fmaf(__uint_as_float(sb[2 * j + 1]), p.scale_log2, neg_mref);
            const int col = c0 + 2 * j;
            if (col < lo || col > hi) a0 = -INFINITY;
            if (col + 1 < lo || col + 1 > hi) a1 = -INFINITY;
            if (col + 32 < lo || col + 32 > hi) b0 = -INFINITY;
            if (col + 33 < lo || col + 33 > hi) b1 = -INFINITY;
            const float p0 = ex2_approx(a0), p1 = ex2_approx(a1), p2 = ex2_approx(b0), p3 = ex2_approx(b1);
            ls[j & 3] += (p0 + p1) + (p2 + p3);
            sa[j] = pack_bf16(p0, p1);
            sb[j] = pack_bf16(p2, p3);
          }
        }
        {
          uint32_t pa[16], pb[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            pa[j] = sa[j];
            pb[j] = sb[j];
          }
          tmem_st16(tS + lane_off + c0, pa);
          tmem_st16(tS + lane_off + c0 + 16, pb);
        }
        l += (ls[0] + ls[1]) + (ls[2] + ls[3]);
        if (tid == 64) WPROF(1, kt, 3);
        tmem_wait_st();
        tc_fence_before_sync();
        mbar_arrive(&p_full);
        if (tid == 64) WPROF(1, kt, 4);
      }
      if (!ok) break;
      // epilogue: O / l -> bf16 -> shared (swizzled; the unit's last V tile is dead once its product
      // is done) -> TMA store; this warp takes its half of the output columns
      l_s[hh][r] = l;
      asm volatile("bar.sync %0, 64;" ::"r"(2 + quarter) : "memory");
      ok = mbar_wait(&o_full, nu & 1, p.status, 32);
      tc_fence_after_sync();
      if (ok) {
        const float inv = 1.f / (l_s[0][r] + l_s[1][r]);
#pragma unroll
        for (int c = 0; c < D / 64; ++c) {
          const int col0 = hh * (D / 2) + c * 32;  // first of 32 output columns
          uint32_t oreg[32];
          tmem_ld32(tO + lane_off + col0, oreg);
          tmem_wait_ld();
          uint8_t* box = sV + (col0 >> 6) * 16384;
#pragma unroll
          for (int g = 0; g < 4; ++g) {  // 4 chunks of 8 columns
            uint4 val;
            val.x = pack_bf16(__uint_as_float(oreg[8 * g + 0]) * inv, __uint_as_float(oreg[8 * g + 1]) * inv);
            val.y = pack_bf16(__uint_as_float(oreg[8 * g + 2]) * inv, __uint_as_float(oreg[8 * g + 3]) * inv);
            val.z = pack_bf16(__uint_as_float(oreg[8 * g + 4]) * inv, __uint_as_float(oreg[8 * g + 5]) * inv);
            val.w = pack_bf16(__uint_as_float(oreg[8 * g + 6]) * inv, __uint_as_float(oreg[8 * g + 7]) * inv);
            *reinterpret_cast<uint4*>(box + swz128_offset(r, (col0 & 63) + g * 8)) = val;
          }
        }
        tc_fence_before_sync();
        fence_proxy_async_smem();
      }
      // every thread has read its part of O and staged it (also the barrier that lets l_s be reused)
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (warp == 2 && elect_one()) {
        mbar_arrive(&o_free);  // the next unit's first product may overwrite O
        if (ok) {
          const uint64_t pol_out = l2_policy_evict_first();  // nobody reads O again
          for (int c = 0; c < D / 64; ++c) tma_store_4d_hint(&mo, sV + c * 16384, c * 64, i0, x.h, x.b, pol_out);
          tma_store_commit();
          tma_store_wait_read<0>();
        }
        mbar_arrive(&v_empty);  // the staging buffer may take the next unit's first V tile
      }
    }
    if (warp == 2 && elect_one()) tma_store_wait_all<0>();
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 256);
}

}  // namespace

#ifdef GF_PROFILE
extern "C" int gformer_debug_read_wprofile(unsigned long long* host_dst) {
  return (int)cudaMemcpyFromSymbol(host_dst, g_wprof, sizeof(g_wprof));
}
#endif

bool tc_window_supported(int N, int d, int w, int dtype) {
  (void)N;
  (void)w;
  return dtype == GF_BF16 && (d == 64 || d == 128);
}

cudaError_t launch_window_tc(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d,
                             int w, int fwd, float scale, int layout, int h_begin, int h_count, WsHeader* ws,
                             cudaStream_t stream) {
  if (h_count <= 0) return cudaSuccess;
  CUtensorMap mq, mk, mv, mo;
  if (!make_qkv_tensor_map(&mq, q, B, H, N, d, layout, 128) || !make_qkv_tensor_map(&mk, k, B, H, N, d, layout, 128) ||
      !make_qkv_tensor_map(&mv, v, B, H, N, d, layout, 128) || !make_qkv_tensor_map(&mo, o, B, H, N, d, layout, 128))
    return cudaErrorInvalidValue;
  WinParams p;
  p.N = N;
  p.w = w;
  p.tiles_back = (w - 1 + 127) / 128;
  p.fwd = fwd;
  p.tiles_fwd = (fwd + 127) / 128;
  p.scale_log2 = scale * kLog2e;
  p.h_begin = h_begin;
  p.h_count = h_count;
  p.nqt = (N + 127) / 128;
  const long long total = (long long)B * h_count * p.nqt;
  if (total > 0x7fffffffLL) return cudaErrorInvalidValue;
  p.total = (int)total;
  p.status = &ws->status;
  p.ticket = &ws->ticket;  // zeroed with the workspace header by the caller
  int dev = 0, sms = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  // persistent CTAs, two per SM; they never wait for one another, so it does not matter how many
  // of them are resident at a time
  dim3 grid((unsigned)(total < 2LL * sms ? total : 2LL * sms));
  auto launch = [&](auto kern, int smem) -> cudaError_t {
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (err != cudaSuccess) return err;
    kern<<<grid, kThreads, smem, stream>>>(mq, mk, mv, mo, p);
    return cudaSuccess;
  };
  if (d == 64)
    e = fwd > 0 ? launch(window_tc_kernel<64, true>, WinSmem<64>::kBytes)
                : launch(window_tc_kernel<64, false>, WinSmem<64>::kBytes);
  else
    e = fwd > 0 ? launch(window_tc_kernel<128, true>, WinSmem<128>::kBytes)
                : launch(window_tc_kernel<128, false>, WinSmem<128>::kBytes);
  if (e != cudaSuccess) return e;
  note_launch();
  return cudaGetLastError();
}

}  // namespace gf
