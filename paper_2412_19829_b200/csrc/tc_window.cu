// Windowed causal softmax attention on the tensor cores (bf16 in, fp32 accumulate).
//
// A work unit is a pair of neighbouring tiles of 128 query rows ("A" and "B") of one (batch, head).
// The keys the two tiles can see, [i0 - w + 1, i0 + 255], overlap almost completely, so every K/V
// tile is loaded once per unit and used by both ("streams").  K and V travel in half tiles of 64
// keys through two TMA rings.  Per stream x and half tile n of its key range:
//   S_x = Q_x K_n^T   tcgen05.mma, A and B from shared memory (K-major), S (128x64 fp32) into one of
//                     the stream's two S buffers in TMEM
//   P_x = softmax     two threads per query row (32 key columns each) read the S row from TMEM, mask
//                     (causal edge on the diagonal tile, window edge on the leftmost ones), agree on
//                     the row maximum through shared memory, exponentiate against a running
//                     reference maximum and write P as bf16 back over S in TMEM
//   O_x += P_x V_n    tcgen05.mma with A = P from TMEM, B = V from shared memory (MN-major)
// With two S buffers the product S(n + 1) runs while the softmax warps work on S(n); with two
// streams the tensor core and the exponential unit always have a second customer.  O stays in TMEM
// across key tiles; it is rescaled only when a row's maximum moves by more than 2^8 (lazy
// rescaling).  Final rows are divided by the softmax denominator, packed to bf16, staged in the
// tile's own (by then dead) Q buffer and written with a TMA store.
// (A 128-key S tile per product would use the tensor core twice as well -- an M = 128 product costs
// about 65 cycles whether N is 64 or 128 -- but TMEM has no room for two of them per stream beside
// O, and with a single S buffer the chain S -> softmax -> P V -> S is serial: measured slower.)
//
// One persistent CTA per SM draws units from a global ticket counter.  Three Q buffers rotate over
// the query tiles a CTA meets, so that a tile's Q is loaded while the two tiles before it are at
// work and a tile's output leaves while the next ones run.  CTAs never wait for one another.
//
// Warp roles: warps 0..15 softmax/epilogue (stream = warp / 8, column half = (warp / 4) % 2, TMEM
// lane quarter = warp % 4), warp 16 = K/V producer (also draws the tickets), warps 17 and 18 = MMA
// issuers of the two streams, warp 19 = Q loads and output stores.
// TMEM: S_A[2] | S_B[2] | O_A | O_B = 512 columns.
#include <type_traits>

#include "common.cuh"
#include "sm100.cuh"

namespace gf {
namespace {

using namespace sm100;

constexpr int kWarpLoad = 16, kWarpMma = 17, kWarpIo = 19;  // warps 0..15: softmax; warps 17 and 18 issue the products
constexpr int kThreads = 20 * 32;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleThreshold = 8.0f;  // log2 units
constexpr int kUnitRing = 8;               // no role is ever this many units behind the producer

__device__ __forceinline__ float ex2_approx(float x) {  // 2^x, flushes denormals, 2^-inf = 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// mbarriers and the unit list, carved from the end of the dynamic shared memory
struct WinCtl {
  uint64_t q_full[3], stage_full[3];                       // per Q buffer
  uint64_t k_full[8], k_empty[8], v_full[8], v_empty[8];   // per ring slot
  uint64_t s_full[2][2], p_full[2][2];             // per query tile of the pair and S buffer
  uint64_t pv_done[2], o_full[2], o_free[2];       // per query tile of the pair
  uint32_t front;  // ring number of the half tile stream 0's next S will read (stream 1 stays behind it)
  uint32_t tmem_base;
  int units_posted;          // entries of unit_ring written so far (monotonic)
  int unit_ring[kUnitRing];  // the CTA's n-th work unit (-1: no more)
};

template <int D>
struct WinSmem {
  static constexpr int kTile = 128 * D * 2;             // bytes of one 128 x D bf16 tile
  static constexpr int kHalf = 64 * D * 2;              // bytes of 64 keys: the unit of the K and V rings
  static constexpr int kStages = (D == 128) ? 4 : 8;    // K and V ring depth, in half tiles
  static constexpr int kX = 0;                          // three Q / output-staging buffers
  static constexpr int kK = 3 * kTile;
  static constexpr int kV = 3 * kTile + kStages * kHalf;
  static constexpr int kMx = 3 * kTile + 2 * kStages * kHalf;  // half-row maxima, bf16 [tile][parity][half][row]
  static constexpr int kCtl = kMx + 2048;
  // d = 128 fills the shared memory of an SM: the tiles must start at the (1024-byte aligned) base
  static constexpr int kSlack = (D == 128) ? 0 : 1024;
  static constexpr int kBytes = kCtl + 640 + kSlack;
};
static_assert(sizeof(WinCtl) <= 640, "control block");
static_assert(WinSmem<128>::kBytes <= 227 * 1024, "shared memory of one SM");

struct WinParams {
  int N, w, tiles_back;  // tiles_back = number of key tiles before the diagonal one
  int fwd, tiles_fwd;    // keys after the query it may see (0: causal; w - 1: two-sided) and the tiles they span
  float scale_log2;
  int h_begin, h_count, nqt, npair, total;  // work units: (batch, head, pair of query tiles), pair fastest
  unsigned int* status;
  unsigned int* ticket;  // zero at launch; units beyond the first one of every CTA come from here
};

// A wait that first polls the barrier for a few microseconds (a thread parked in try_wait takes a
// few hundred cycles to come back) and then falls back to the bounded parked wait.
__device__ __forceinline__ bool mbar_wait_hot(uint64_t* bar, uint32_t parity, unsigned int* status,
                                              unsigned int where) {
#pragma unroll 1
  for (int it = 0; it < 2000; ++it)
    if (mbar_test_wait(bar, parity)) return true;
  return mbar_wait(bar, parity, status, where);
}

// Bounded poll of a monotonic counter in shared memory.
__device__ __forceinline__ bool win_wait_epoch(const int* counter, int target, unsigned int* status,
                                               unsigned int where) {
  const volatile int* c = counter;
  if (*c >= target) { __threadfence_block(); return true; }
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

// A unit: query tiles qtA (and qtA + 1 when nt == 2); tile x walks the key tiles f[x] .. l[x].
struct Unit {
  int h, b, qtA, nt;
  int f[2], l[2];
};

template <int D, bool kTwoSided>
__global__ void __launch_bounds__(kThreads, 1)
window_tc_kernel(const __grid_constant__ CUtensorMap mq, const __grid_constant__ CUtensorMap mk,
                 const __grid_constant__ CUtensorMap mv, const __grid_constant__ CUtensorMap mo,
                 const WinParams p) {
  using SM = WinSmem<D>;
  constexpr int ST = SM::kStages;
  extern __shared__ __align__(1024) uint8_t raw_smem[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(raw_smem) + 1023) & ~(uintptr_t)1023);
  if (sm + SM::kCtl + 640 > raw_smem + SM::kBytes) {  // misaligned base with no slack: report, do nothing
    if (threadIdx.x == 0 && atomicCAS(p.status, 0u, 1u) == 0u) p.status[1] = 99;
    return;
  }
  uint8_t* sX = sm + SM::kX;
  uint8_t* sK = sm + SM::kK;
  uint8_t* sV = sm + SM::kV;
  __nv_bfloat16* mx_s = reinterpret_cast<__nv_bfloat16*>(sm + SM::kMx);
  WinCtl* ctl = reinterpret_cast<WinCtl*>(sm + SM::kCtl);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int i = 0; i < 3; ++i) {
      mbar_init(&ctl->q_full[i], 1);
      mbar_init(&ctl->stage_full[i], 256);
    }
    for (int i = 0; i < 8; ++i) {
      mbar_init(&ctl->k_full[i], 1);
      mbar_init(&ctl->k_empty[i], 2);  // one arrival per stream
      mbar_init(&ctl->v_full[i], 1);
      mbar_init(&ctl->v_empty[i], 2);
    }
    for (int i = 0; i < 2; ++i) {
      for (int b = 0; b < 2; ++b) {
        mbar_init(&ctl->s_full[i][b], 1);
        mbar_init(&ctl->p_full[i][b], 256);
      }
      mbar_init(&ctl->pv_done[i], 1);
      mbar_init(&ctl->o_full[i], 1);
      mbar_init(&ctl->o_free[i], 256);
    }
    ctl->unit_ring[0] = blockIdx.x;  // the grid never exceeds the number of units
    ctl->front = 0;
    ctl->units_posted = 1;
    mbar_fence_init();
    tma_prefetch_desc(&mq);
    tma_prefetch_desc(&mk);
    tma_prefetch_desc(&mv);
    tma_prefetch_desc(&mo);
  }
  if (warp == kWarpMma) {
    tmem_alloc(&ctl->tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = ctl->tmem_base;

  auto decode = [&](int u) {
    Unit x;
    const int pq = u % p.npair;
    const int bh = u / p.npair;
    x.h = p.h_begin + bh % p.h_count;
    x.b = bh / p.h_count;
    x.qtA = 2 * pq;
    x.nt = (x.qtA + 1 < p.nqt) ? 2 : 1;
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      const int qt = x.qtA + t;
      x.f[t] = (qt - p.tiles_back) > 0 ? (qt - p.tiles_back) : 0;
      // kTwoSided: the tiles after the diagonal one that the window reaches, up to the sequence end
      x.l[t] = !kTwoSided ? qt : ((qt + p.tiles_fwd) < p.nqt ? (qt + p.tiles_fwd) : p.nqt - 1);
    }
    return x;
  };
  auto unit_at = [&](uint32_t n) -> int {
    if (!win_wait_epoch(&ctl->units_posted, (int)n + 1, p.status, 90)) return -1;
    return reinterpret_cast<const volatile int*>(ctl->unit_ring)[n % kUnitRing];
  };

  // Every role walks the same list of units and keeps the same running counters (units, query
  // tiles, key tiles), from which the ring slots and barrier phases follow.
  if (warp == kWarpLoad) {
    // ------------------------------------------------------------ K/V producer + ticket drawer
    if (elect_one()) {
      uint32_t nu = 0, kt = 0;
      bool ok = true;
      for (int u = blockIdx.x; u >= 0 && ok;) {
        const Unit x = decode(u);
        // draw the next ticket now; its value is needed once this unit's first loads are out
        const unsigned int t_next = atomicAdd(p.ticket, 1u);
        int u_next = -1;
        const int g0 = x.f[0], g1 = x.nt == 2 ? x.l[1] : x.l[0];
        for (int hg = 2 * g0; hg <= 2 * g1 + 1; ++hg, ++kt) {  // kt counts half tiles here
          const uint32_t slot = kt % ST, use = kt / ST;
          if (use >= 1 && !mbar_wait(&ctl->k_empty[slot], (use - 1) & 1, p.status, 10)) { ok = false; break; }
          mbar_arrive_expect_tx(&ctl->k_full[slot], SM::kHalf);
          for (int c = 0; c < D / 64; ++c)
            tma_load_4d(sK + slot * SM::kHalf + c * 8192, &mk, &ctl->k_full[slot], c * 64, hg * 64, x.h, x.b);
          if (use >= 1 && !mbar_wait(&ctl->v_empty[slot], (use - 1) & 1, p.status, 11)) { ok = false; break; }
          mbar_arrive_expect_tx(&ctl->v_full[slot], SM::kHalf);
          for (int c = 0; c < D / 64; ++c)
            tma_load_4d(sV + slot * SM::kHalf + c * 8192, &mv, &ctl->v_full[slot], c * 64, hg * 64, x.h, x.b);
          if (hg == 2 * g0) {  // the other roles learn of the next unit early (its Q is requested ahead)
            u_next = (t_next < (unsigned int)(p.total - (int)gridDim.x)) ? (int)(gridDim.x + t_next) : -1;
            ctl->unit_ring[(nu + 1) % kUnitRing] = u_next;
            __threadfence_block();
            *reinterpret_cast<volatile int*>(&ctl->units_posted) = (int)nu + 2;
          }
        }
        ++nu;
        u = u_next;
      }
    }
  } else if (warp == kWarpIo) {
    // ------------------------------------------------------------ Q loads and output stores
    // Query tile number n of this CTA lives in buffer n % 3: its Q lands there, its output is staged
    // there, and once the store has read it the buffer takes the Q of tile n + 3.
    if (elect_one()) {
      const uint64_t pol_once = l2_policy_evict_first();  // Q is read once, nobody reads O again
      uint32_t ld_nu = 0, ql = 0, st_nu = 0, qs = 0;
      int ld_which = 0, st_which = 0;
      bool ld_end = false;
      auto load_next = [&]() {
        if (ld_end) return;
        const int u = unit_at(ld_nu);
        if (u < 0) { ld_end = true; return; }
        const Unit x = decode(u);
        const uint32_t buf = ql % 3;
        mbar_arrive_expect_tx(&ctl->q_full[buf], SM::kTile);
        for (int c = 0; c < D / 64; ++c)
          tma_load_4d_hint(sX + buf * SM::kTile + c * 16384, &mq, &ctl->q_full[buf], c * 64,
                           (x.qtA + ld_which) * 128, x.h, x.b, pol_once);
        ++ql;
        if (++ld_which == x.nt) { ld_which = 0; ++ld_nu; }
      };
      load_next();
      load_next();
      load_next();
      for (;;) {
        const int u = unit_at(st_nu);
        if (u < 0) break;
        const Unit x = decode(u);
        const uint32_t buf = qs % 3;
        if (!mbar_wait(&ctl->stage_full[buf], (qs / 3) & 1, p.status, 40)) break;
        for (int c = 0; c < D / 64; ++c)
          tma_store_4d_hint(&mo, sX + buf * SM::kTile + c * 16384, c * 64, (x.qtA + st_which) * 128, x.h, x.b,
                            pol_once);
        tma_store_commit();
        tma_store_wait_read<0>();
        ++qs;
        if (++st_which == x.nt) { st_which = 0; ++st_nu; }
        load_next();
      }
      tma_store_wait_all<0>();
    }
  } else if (warp == kWarpMma || warp == kWarpMma + 1) {
    // ------------------------------------------------------------ MMA issuers
    // One issuing thread per query tile of the pair ("stream").  A stream's products are, in order,
    // S(0), S(1), then P V(j) followed by S(j + 2): S buffer j & 1 is free again once P V(j) has been
    // issued, because the tensor core runs one thread's products in issue order.  The two streams
    // meet only in the ring: a half tile goes back to the producer when both streams are done
    // with it, and stream 1, whose window starts one key tile later, does not overtake stream 0,
    // so that the two read the same half tile at about the same time and the rest of the ring
    // holds loads in flight.
    if (elect_one()) {
      constexpr uint32_t idesc_qk = umma_idesc_bf16(128, 64, false, false);
      constexpr uint32_t idesc_pv = umma_idesc_bf16(128, D, false, true);
      const uint32_t aX = smem_u32(sX), aK = smem_u32(sK), aV = smem_u32(sV);
      auto run_stream = [&](auto T) {
        constexpr int t = decltype(T)::value;
        const uint32_t tSt = tmem + t * 128, tO = tmem + 256 + t * D;
        volatile uint32_t* front = &ctl->front;
        uint32_t kt = 0, qn = 0, sub = 0, ntile = 0;  // key tiles, query tiles (both streams), own sub-tiles and tiles so far
        for (uint32_t nu = 0;; ++nu) {
          const int u = unit_at(nu);
          if (u < 0) break;
          const Unit x = decode(u);
          const int g0 = x.f[0];
          const int n_key = (x.nt == 2 ? x.l[1] : x.l[0]) - g0 + 1;
          // The stream walks every half tile of the unit in ring order, for S and (two steps behind)
          // for P V.  Half tiles outside its own key range it only hands on: it waits until they
          // have landed and arrives on their release barrier.  That way every thread that waits on
          // a slot sees each of its phases exactly once, in order (a parity wait tells a barrier's
          // current phase only from the one before it), and a slot is released by exactly two
          // arrivals whoever reads it.
          const bool mine = t < x.nt;
          const int off = mine ? 2 * (x.f[t] - g0) : 0;  // own sub-tile j is half tile off + j of the unit
          const int n_sub = mine ? 2 * (x.l[t] - x.f[t] + 1) : 0;
          const uint32_t rbase = 2 * kt;  // ring number of the unit's first half tile
          const uint32_t qbuf = (qn + t) % 3;
          const uint32_t qa = aX + qbuf * SM::kTile;
          for (int m = 0; m < 2 * n_key + 2; ++m) {
            if (m >= 2) {
              const int jj = m - 2 - off;
              const uint32_t n = rbase + (uint32_t)(m - 2), slot = n % ST;
              if (!mbar_wait(&ctl->v_full[slot], (n / ST) & 1, p.status, 23)) return;
              if (jj >= 0 && jj < n_sub) {  // O += P V of sub-tile jj
                const int half = jj & 1;
                if (!mbar_wait_hot(&ctl->p_full[t][half], ((sub + jj) >> 1) & 1, p.status, 22)) return;
                // the first product of a tile overwrites O: the previous tile's epilogue has read it
                if (jj == 0 && ntile >= 1 && !mbar_wait(&ctl->o_free[t], (ntile - 1) & 1, p.status, 24)) return;
                tc_fence_after_sync();
                const uint32_t va = aV + slot * SM::kHalf, tP = tSt + half * 64;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                  umma_ts(tO, tP + (ks >> 1) * 32 + (ks & 1) * 8, umma_smem_desc(va + ks * 2048, 8192, 1024), idesc_pv,
                          (jj > 0) || (ks > 0));
                umma_commit(&ctl->v_empty[slot]);
                umma_commit(&ctl->pv_done[t]);
                if (jj == n_sub - 1) umma_commit(&ctl->o_full[t]);
              } else {
                mbar_arrive(&ctl->v_empty[slot]);
              }
            }
            if (m < 2 * n_key) {
              const int j = m - off;
              const uint32_t n = rbase + (uint32_t)m, slot = n % ST;
              if (j >= 0 && j < n_sub) {  // S of sub-tile j into S buffer j & 1
                const int half = j & 1;
                if (t == 1) {  // bounded: stream 0's next S must lie behind this half tile
                  if (*front <= n) {
                    const long long t0 = clock64(), limit = wait_limit_cycles(p.status);
                    while (*front <= n) {
                      if (clock64() - t0 > limit) {
                        if (atomicCAS(p.status, 0u, 1u) == 0u) p.status[1] = 26;
                        return;
                      }
                      __nanosleep(20);
                    }
                  }
                }
                if (j == 0 && !mbar_wait(&ctl->q_full[qbuf], ((qn + t) / 3) & 1, p.status, 20)) return;
                if (!mbar_wait(&ctl->k_full[slot], (n / ST) & 1, p.status, 21)) return;
                tc_fence_after_sync();
                const uint32_t ka = aK + slot * SM::kHalf;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks)
                  umma_ss(tSt + half * 64, umma_smem_desc(qa + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024),
                          umma_smem_desc(ka + (ks >> 2) * 8192 + (ks & 3) * 32, 16, 1024), idesc_qk, ks > 0);
                umma_commit(&ctl->s_full[t][half]);
                umma_commit(&ctl->k_empty[slot]);
                // stream 0 tells where its next S will read: the next half tile of this query tile,
                // or the first one of the next unit
                if (t == 0) *front = (j + 1 < n_sub) ? n + 1 : 2 * (kt + (uint32_t)n_key);
              } else {
                if (!mbar_wait(&ctl->k_full[slot], (n / ST) & 1, p.status, 21)) return;
                mbar_arrive(&ctl->k_empty[slot]);
              }
            }
          }
          if (mine) {
            sub += (uint32_t)n_sub;
            ++ntile;
          }
          kt += (uint32_t)n_key;
          qn += (uint32_t)x.nt;
        }
        if (t == 0) *front = 0xffffffffu;
      };
      if (warp == kWarpMma)
        run_stream(std::integral_constant<int, 0>{});
      else
        run_stream(std::integral_constant<int, 1>{});
    }
  } else {
    // ------------------------------------------------------------ softmax + epilogue
    // Two threads per query row, 64 key columns of a tile each (four warps per scheduler hide one
    // another's latencies and keep the exponential unit fed).
    const int t = warp >> 3;         // query tile of the pair
    const int hh = (warp >> 2) & 1;  // half of the key columns (softmax) / of the output columns (epilogue)
    const int quarter = warp & 3;    // TMEM lane quarter this warp may touch
    const int r = quarter * 32 + lane;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const uint32_t tO = tmem + 256 + t * D + lane_off;
    const int pair_bar = 1 + t * 4 + quarter;  // named barrier of the two warps that share 32 rows
    uint32_t nu = 0, sub = 0, ntile = 0, qn = 0;
    bool ok = true;
    for (; ok; ++nu) {
      const int u = unit_at(nu);
      if (u < 0) break;
      const Unit x = decode(u);
      const uint32_t buf = (qn + t) % 3;
      qn += (uint32_t)x.nt;
      if (t >= x.nt) continue;
      const int i0 = (x.qtA + t) * 128, i = i0 + r;
      const int f_t = t ? x.f[1] : x.f[0], l_t = t ? x.l[1] : x.l[0];  // (no run-time index: the unit stays in registers)
      const int n_sub = 2 * (l_t - f_t + 1);
      const int i_first = i0 + quarter * 32;  // the warp's first row
      float m_ref = -INFINITY;  // reference maximum the stored O and l are relative to (same in both halves)
      float l = 0.f;            // sum over this thread's columns
      for (int j = 0; j < n_sub; ++j, ++sub) {
        const int half = j & 1;  // which 64 keys of the key tile; also the S buffer
        const int j0 = (f_t + (j >> 1)) * 128 + half * 64 + hh * 32;  // first key of this thread's 32 columns
        const uint32_t tS = tmem + t * 128 + half * 64 + hh * 32 + lane_off;
        // valid key columns of this row among its 32: [lo, hi]; over the warp's 32 rows lo and hi move
        // by 31, so the block is classified per warp: nothing visible (costs nothing), all visible to
        // every row (no per-element test), or mixed
        const int lo = i - p.w + 1 - j0;
        // (two-sided window: the query also sees p.fwd keys after it, and keys past the end do not exist)
        const int hi = kTwoSided ? min(i + p.fwd, p.N - 1) - j0 : i - j0;
        const int lo_first = i_first - p.w + 1 - j0;  // lo of the warp's first row (last row: +31)
        const int hi_first = kTwoSided ? min(i_first + p.fwd, p.N - 1) - j0 : i_first - j0;  // hi of its first row
        const int hi_last = kTwoSided ? min(i_first + 31 + p.fwd, p.N - 1) - j0 : hi_first + 31;  // ... of its last row
        const bool none = (31 < lo_first || 0 > hi_last);
        const bool inside = (0 >= lo_first + 31) && (31 <= hi_first);
        if (!mbar_wait_hot(&ctl->s_full[t][half], (sub >> 1) & 1, p.status, 30)) { ok = false; break; }
        tc_fence_after_sync();
        // the block's 32 scores stay in registers from the maximum to the exponentials
        uint32_t sa[32];
        float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        if (!none) {
          tmem_ld32(tS, sa);
          tmem_wait_ld();
          if (!inside) {
#pragma unroll
            for (int c = 0; c < 32; ++c)
              if (c < lo || c > hi) sa[c] = 0xff800000u;  // -inf
          }
#pragma unroll
          for (int c = 0; c < 32; ++c) mx[c & 3] = fmaxf(mx[c & 3], __uint_as_float(sa[c]));
        }
        // the row maximum over both halves: exchange through shared memory with the partner warp
        // (same lane quarter, other half); double buffered by sub-tile parity, one barrier per sub-tile.
        // The halves exchange bf16 values rounded up, and both use the rounded pair, so that they
        // agree on the reference bit for bit (a reference slightly above the maximum is as good).
        const __nv_bfloat16 mloc = __float2bfloat16_ru(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])));
        __nv_bfloat16* mx_row = mx_s + ((t * 2 + half) * 2) * 128 + r;
        mx_row[hh * 128] = mloc;
        asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
        const float mt = fmaxf(__bfloat162float(mloc), __bfloat162float(mx_row[(hh ^ 1) * 128])) * p.scale_log2;  // scale > 0
        // lazy rescale of what has been accumulated so far (both halves take the same decision)
        float alpha = 1.f;
        bool need = false;
        if (mt > m_ref + kRescaleThreshold) {  // also true for the first finite maximum
          need = (m_ref != -INFINITY);         // nothing accumulated yet otherwise (O row and l are 0)
          alpha = need ? exp2f(m_ref - mt) : 1.f;
          m_ref = mt;
          l *= alpha;
        }
        if (j > 0) {
          if (__any_sync(0xffffffffu, need)) {
            // every product issued so far has to be in O (the S product of this sub-tile was issued
            // behind all but the last of them, so at most that one is still running)
            if (!mbar_wait(&ctl->pv_done[t], (sub - 1) & 1, p.status, 31)) { ok = false; break; }
            tc_fence_after_sync();
            // this warp's half of the output columns, a few at a time (rare path)
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
              uint32_t oreg[16];
              tmem_ld16(tO + hh * (D / 2) + c * 16, oreg);
              tmem_wait_ld();
#pragma unroll
              for (int e = 0; e < 16; ++e) oreg[e] = __float_as_uint(__uint_as_float(oreg[e]) * alpha);
              tmem_st16(tO + hh * (D / 2) + c * 16, oreg);
            }
            tmem_wait_st();
          }
        }
        // p = 2^(s * scale_log2 - m_ref), bf16, back over S: this thread's 32 scores become 16 packed
        // columns at the start of the columns it has itself consumed
        const float neg_mref = (m_ref == -INFINITY) ? 0.f : -m_ref;
        float ls[4] = {0.f, 0.f, 0.f, 0.f};
        uint32_t pa[16];
        if (none) {
#pragma unroll
          for (int c = 0; c < 16; ++c) pa[c] = 0u;
        } else {  // masked scores are -inf: their exponentials are 0
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            const float p0 = ex2_approx(fmaf(__uint_as_float(sa[2 * c]), p.scale_log2, neg_mref));
            const float p1 = ex2_approx(fmaf(__uint_as_float(sa[2 * c + 1]), p.scale_log2, neg_mref));
            ls[c & 3] += p0 + p1;
            pa[c] = pack_bf16(p0, p1);
          }
        }
        tmem_st16(tS, pa);
        l += (ls[0] + ls[1]) + (ls[2] + ls[3]);
        tmem_wait_st();
        tc_fence_before_sync();
        mbar_arrive(&ctl->p_full[t][half]);
      }
      if (!ok) break;
      // epilogue: O / l -> bf16 -> shared (swizzled; the tile's Q buffer is dead once its last product
      // is done) -> TMA store by the store warp; this warp takes its half of the output columns
      ok = mbar_wait(&ctl->o_full[t], ntile & 1, p.status, 32);
      if (!ok) break;
      tc_fence_after_sync();
      uint8_t* stage = sX + buf * SM::kTile;
      // the two halves of a row add their sums through bytes of the staging buffer that the
      // writing thread itself will later overwrite with output
      {
        const int mine = hh * (D / 2), theirs = (hh ^ 1) * (D / 2);
        *reinterpret_cast<float*>(stage + (mine >> 6) * 16384 + swz128_offset(r, mine & 63)) = l;
        asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
        const float lp = *reinterpret_cast<const float*>(stage + (theirs >> 6) * 16384 + swz128_offset(r, theirs & 63));
        asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
        l = hh == 0 ? l + lp : lp + l;
      }
      const float inv = 1.f / l;
#pragma unroll
      for (int c = 0; c < D / 64; ++c) {
        const int col0 = hh * (D / 2) + c * 32;  // first of 32 output columns
        uint32_t oreg[32];
        tmem_ld32(tO + col0, oreg);
        tmem_wait_ld();
        uint8_t* box = stage + (col0 >> 6) * 16384;
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
      mbar_arrive(&ctl->o_free[t]);  // the slot's next tile may overwrite O
      fence_proxy_async_smem();
      mbar_arrive(&ctl->stage_full[buf]);  // the store warp ships the tile
      ++ntile;
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kWarpMma) tmem_dealloc(tmem, 512);
}

}  // namespace

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
  if (!make_qkv_tensor_map(&mq, q, B, H, N, d, layout, 128) || !make_qkv_tensor_map(&mk, k, B, H, N, d, layout, 64) ||
      !make_qkv_tensor_map(&mv, v, B, H, N, d, layout, 64) || !make_qkv_tensor_map(&mo, o, B, H, N, d, layout, 128))
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
  p.npair = (p.nqt + 1) / 2;
  const long long total = (long long)B * h_count * p.npair;
  if (total > 0x7fffffffLL) return cudaErrorInvalidValue;
  p.total = (int)total;
  p.status = &ws->status;
  p.ticket = &ws->ticket;  // zeroed with the workspace header by the caller
  int dev = 0, sms = 0;
  cudaError_t e;
  if ((e = device_info(&dev, &sms)) != cudaSuccess) return e;
  // one persistent CTA per SM (it takes the SM's whole tensor memory); CTAs never wait for one
  // another, so it does not matter how many of them are resident at a time
  dim3 grid((unsigned)(total < sms ? total : sms));
  auto launch = [&](auto kern, int smem) -> cudaError_t {
    cudaError_t err = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), dev, smem);
    if (err != cudaSuccess) return err;
    kern<<<grid, kThreads, smem, stream>>>(mq, mk, mv, mo, p);
    return cudaSuccess;
  };
  if (d == 64)
    e = fwd > 0 ? launch(window_tc_kernel<64, true>, WinSmem<64>::kBytes) : launch(window_tc_kernel<64, false>, WinSmem<64>::kBytes);
  else
    e = fwd > 0 ? launch(window_tc_kernel<128, true>, WinSmem<128>::kBytes)
                : launch(window_tc_kernel<128, false>, WinSmem<128>::kBytes);
  if (e != cudaSuccess) return e;
  note_launch();
  return cudaGetLastError();
}

}  // namespace gf
