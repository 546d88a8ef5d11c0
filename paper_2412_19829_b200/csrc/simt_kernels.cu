// CUDA-core (fp32 arithmetic) kernels of libgformer.
//
// They serve every request the tensor-core kernels do not take: fp32 storage, windows
// that are not a multiple of 64, and the memory-bound decode step / ring export, which
// have no dense contraction worth a tensor core.  All of them are plain data-parallel
// kernels: no inter-CTA communication, no spin waits.
#include "common.cuh"

namespace gf {
namespace {

template <typename T> struct Vec4;
template <> struct Vec4<float> {
  static __device__ __forceinline__ float4 load(const float* p) { return *reinterpret_cast<const float4*>(p); }
  static __device__ __forceinline__ void store(float* p, float4 x) { *reinterpret_cast<float4*>(p) = x; }
};
template <> struct Vec4<__nv_bfloat16> {
  static __device__ __forceinline__ float4 load(const __nv_bfloat16* p) {
    uint2 raw = *reinterpret_cast<const uint2*>(p);
    __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&raw.x);
    __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&raw.y);
    float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
    return make_float4(fa.x, fa.y, fb.x, fb.y);
  }
  static __device__ __forceinline__ void store(__nv_bfloat16* p, float4 x) {
    __nv_bfloat162 a = __floats2bfloat162_rn(x.x, x.y);
    __nv_bfloat162 b = __floats2bfloat162_rn(x.z, x.w);
    uint2 raw;
    raw.x = *reinterpret_cast<uint32_t*>(&a);
    raw.y = *reinterpret_cast<uint32_t*>(&b);
    *reinterpret_cast<uint2*>(p) = raw;
  }
};

// ------------------------------------------------------------------------------------
// Windowed softmax attention (Eq. 1 + causal mask + left window of w keys).
// One CTA = 32 query rows of one head, 4 threads per row, each owning d/4 of the head
// dimension; keys/values pass through shared memory 32 rows at a time; online softmax.
// ------------------------------------------------------------------------------------
template <typename T, int D>
__global__ void __launch_bounds__(128)
window_simt_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                   T* __restrict__ o, int N, int w, int fwd, float scale, Strides st, int h_begin) {
  // fwd: keys after the query that it may see (0: the causal window; w - 1: the two-sided one)
  constexpr int CH = D / 16;  // float4 chunks per thread
  __shared__ __align__(16) float Ks[32][D];
  __shared__ __align__(16) float Vs[32][D];

  const int b = blockIdx.z, h = h_begin + blockIdx.y;
  const long long base = (long long)b * st.b + (long long)h * st.h;
  const int i0 = blockIdx.x * 32;
  const int row = threadIdx.x >> 2, sub = threadIdx.x & 3;
  const int i = i0 + row;

  float4 qv[CH], ov[CH];
#pragma unroll
  for (int c = 0; c < CH; ++c) {
    ov[c] = make_float4(0.f, 0.f, 0.f, 0.f);
    qv[c] = (i < N) ? Vec4<T>::load(q + base + (long long)i * st.n + 4 * (sub + 4 * c))
                    : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  float m = -INFINITY, l = 0.f;

  int jlo = i0 - w + 1;
  if (jlo < 0) jlo = 0;
  int jhi = i0 + 31 + fwd;
  if (jhi > N - 1) jhi = N - 1;

  for (int j0 = jlo; j0 <= jhi; j0 += 32) {
    __syncthreads();
    for (int idx = threadIdx.x; idx < 32 * (D / 4); idx += 128) {
      const int r = idx / (D / 4), c4 = idx % (D / 4);
      const int j = j0 + r;
      float4 kk = make_float4(0.f, 0.f, 0.f, 0.f), vv = kk;
      if (j < N) {
        kk = Vec4<T>::load(k + base + (long long)j * st.n + 4 * c4);
        vv = Vec4<T>::load(v + base + (long long)j * st.n + 4 * c4);
      }
      *reinterpret_cast<float4*>(&Ks[r][4 * c4]) = kk;
      *reinterpret_cast<float4*>(&Vs[r][4 * c4]) = vv;
    }
    __syncthreads();
#pragma unroll 4
    for (int jj = 0; jj < 32; ++jj) {
      const int j = j0 + jj;
      float s = 0.f;
#pragma unroll
      for (int c = 0; c < CH; ++c) {
        const float4 kk = *reinterpret_cast<const float4*>(&Ks[jj][4 * (sub + 4 * c)]);
        s += qv[c].x * kk.x + qv[c].y * kk.y + qv[c].z * kk.z + qv[c].w * kk.w;
      }
      s += __shfl_xor_sync(0xffffffffu, s, 1);
      s += __shfl_xor_sync(0xffffffffu, s, 2);
      const bool valid = (i < N) && (j <= i + fwd) && (j > i - w) && (j < N);
      if (valid) {
        s *= scale;
        const float m_new = fmaxf(m, s);
        const float corr = expf(m - m_new);
        const float p = expf(s - m_new);
        l = l * corr + p;
#pragma unroll
        for (int c = 0; c < CH; ++c) {
          const float4 vv = *reinterpret_cast<const float4*>(&Vs[jj][4 * (sub + 4 * c)]);
          ov[c].x = ov[c].x * corr + p * vv.x;
          ov[c].y = ov[c].y * corr + p * vv.y;
          ov[c].z = ov[c].z * corr + p * vv.z;
          ov[c].w = ov[c].w * corr + p * vv.w;
        }
        m = m_new;
      }
    }
  }
  if (i < N) {
    const float inv = 1.f / l;
#pragma unroll
    for (int c = 0; c < CH; ++c) {
      float4 r = make_float4(ov[c].x * inv, ov[c].y * inv, ov[c].z * inv, ov[c].w * inv);
      Vec4<T>::store(o + base + (long long)i * st.n + 4 * (sub + 4 * c), r);
    }
  }
}

// ------------------------------------------------------------------------------------
// Causal linear attention, Algorithm 1 token by token.
// One CTA = one head x one slice of 32 value columns.  Warp g owns features
// a in [g*D/8, (g+1)*D/8); lane c owns value column c of the slice.  S lives in registers
// (D/8 per thread), z is replicated per lane.  Tokens are staged 16 at a time.
// global_sum != 0: the unmasked form of the bidirectional layer (Sec. II-B) -- a first sweep over
// the tokens only accumulates S and z, a second one only reads them out.
// ------------------------------------------------------------------------------------
template <typename T, int D>
__global__ void __launch_bounds__(256)
linear_simt_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                   T* __restrict__ o, int N, Strides st, int h_begin, int h_count,
                   float* __restrict__ S_io, float* __restrict__ z_io, int zero_init, int global_sum,
                   const T* __restrict__ W /* [h_count, D, D] or null: elu + 1 */) {
  constexpr int TB = 16;
  constexpr int AR = D / 8;
  __shared__ float qs[TB][D];
  __shared__ float ks[TB][D];
  __shared__ float xr[TB][D + 1];  // raw rows while the positive random features are taken (W != null)
  __shared__ float vs[TB][32];
  __shared__ float red[TB][8][33];
  __shared__ float redden[TB][8];

  const int slice = blockIdx.x, hl = blockIdx.y, b = blockIdx.z;
  const int h = h_begin + hl;
  const long long base = (long long)b * st.b + (long long)h * st.h;
  const int tid = threadIdx.x, c = tid & 31, g = tid >> 5;
  const long long sidx = (long long)b * h_count + hl;

  float S[AR], zr[AR];
#pragma unroll
  for (int a = 0; a < AR; ++a) {
    S[a] = 0.f;
    zr[a] = 0.f;
  }
  if (S_io != nullptr && !zero_init) {
#pragma unroll
    for (int a = 0; a < AR; ++a) {
      S[a] = S_io[(sidx * D + (g * AR + a)) * D + slice * 32 + c];
      zr[a] = z_io[sidx * D + g * AR + a];
    }
  }

  for (int sweep = global_sum ? 0 : 1; sweep < 2; ++sweep) {
  const bool accumulate = !global_sum || sweep == 0, readout = !global_sum || sweep == 1;
  for (int n0 = 0; n0 < N; n0 += TB) {
    __syncthreads();
    if (W == nullptr) {
      for (int idx = tid; idx < TB * D; idx += 256) {
        const int tok = idx / D, a = idx % D;
        const int n = n0 + tok;
        float qq = 0.f, kk = 0.f;
        if (n < N) {
          qq = phi_elu1(to_f32(q[base + (long long)n * st.n + a]));
          kk = phi_elu1(to_f32(k[base + (long long)n * st.n + a]));
        }
        qs[tok][a] = qq;
        ks[tok][a] = kk;  // 0 for rows past N: they must not enter the state
      }
    } else {
      // phi_W(x)[a] = exp(<w_a, x> - |x|^2 / 2) / sqrt(D) (Sec. III-A / III-C), Q rows first, then K rows.
      // A factor common to all features of a query cancels in the output: the query features are taken
      // relative to the row's largest projection, exp(<w_a, q> - max_a <w_a, q>), which keeps their
      // products with the state inside the range of fp32.
      const T* Wh = W + (long long)hl * D * D;
      for (int which = 0; which < 2; ++which) {
        const T* src = which ? k : q;
        float (*dst)[D] = which ? ks : qs;
        for (int idx = tid; idx < TB * D; idx += 256) {
          const int tok = idx / D, a = idx % D;
          const int n = n0 + tok;
          xr[tok][a] = (n < N) ? to_f32(src[base + (long long)n * st.n + a]) : 0.f;
        }
        __syncthreads();
        for (int idx = tid; idx < TB * D; idx += 256) {
          const int tok = idx / D, a = idx % D;
          float proj = 0.f, n2 = 0.f;
          for (int cc = 0; cc < D; ++cc) {
            const float x = xr[tok][cc];
            proj = fmaf(to_f32(Wh[(long long)a * D + cc]), x, proj);
            n2 = fmaf(x, x, n2);
          }
          if (which) dst[tok][a] = (n0 + tok < N) ? expf(proj - 0.5f * n2) * rsqrtf((float)D) : 0.f;
          else dst[tok][a] = proj;
        }
        __syncthreads();
        if (which == 0) {  // queries: relative to the row maximum
          float e[TB * D / 256];
          for (int i = 0; i < TB * D / 256; ++i) {
            const int idx = tid + 256 * i, tok = idx / D, a = idx % D;
            float mx = -INFINITY;
            for (int cc = 0; cc < D; ++cc) mx = fmaxf(mx, qs[tok][cc]);
            e[i] = expf(qs[tok][a] - mx);
          }
          __syncthreads();
          for (int i = 0; i < TB * D / 256; ++i) {
            const int idx = tid + 256 * i;
            qs[idx / D][idx % D] = e[i];
          }
          __syncthreads();
        }
      }
    }
    for (int idx = tid; idx < TB * 32; idx += 256) {
      const int tok = idx >> 5, cc = idx & 31;
      const int n = n0 + tok;
      vs[tok][cc] = (n < N) ? to_f32(v[base + (long long)n * st.n + slice * 32 + cc]) : 0.f;
    }
    __syncthreads();
#pragma unroll 1
    for (int tok = 0; tok < TB; ++tok) {
      const float vv = vs[tok][c];
      float num = 0.f, den = 0.f;
#pragma unroll
      for (int a = 0; a < AR; ++a) {
        const float kk = accumulate ? ks[tok][g * AR + a] : 0.f;
        const float qq = qs[tok][g * AR + a];
        S[a] = fmaf(kk, vv, S[a]);
        zr[a] += kk;
        num = fmaf(qq, S[a], num);
        den = fmaf(qq, zr[a], den);
      }
      red[tok][g][c] = num;
      if (c == 0) redden[tok][g] = den;
    }
    __syncthreads();
    for (int idx = tid; idx < TB * 32; idx += 256) {
      const int tok = idx >> 5, cc = idx & 31;
      const int n = n0 + tok;
      float num = 0.f, den = 0.f;
#pragma unroll
      for (int gg = 0; gg < 8; ++gg) {
        num += red[tok][gg][cc];
        den += redden[tok][gg];
      }
      if (n < N && readout) o[base + (long long)n * st.n + slice * 32 + cc] = from_f32<T>(num / den);
    }
  }
  }
  if (S_io != nullptr) {
#pragma unroll
    for (int a = 0; a < AR; ++a) {
      S_io[(sidx * D + (g * AR + a)) * D + slice * 32 + c] = S[a];
      if (slice == 0 && c == 0) z_io[sidx * D + g * AR + a] = zr[a];
    }
  }
}

// ------------------------------------------------------------------------------------
// Ring export: the last min(N, w) keys/values of the windowed heads into slot j mod w.
// ------------------------------------------------------------------------------------
template <typename T>
__global__ void export_ring_kernel(const T* __restrict__ k, const T* __restrict__ v, T* __restrict__ kc,
                                   T* __restrict__ vc, int N, int d, int w, int wn, Strides st,
                                   int h_sparse, long long total4) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total4) return;
  const int d4 = d / 4;
  const int c4 = (int)(idx % d4);
  long long r = idx / d4;
  const int jj = (int)(r % wn);
  r /= wn;
  const int h = (int)(r % h_sparse);
  const int b = (int)(r / h_sparse);
  const int j = N - wn + jj;
  const long long src = (long long)b * st.b + (long long)h * st.h + (long long)j * st.n + 4 * c4;
  const long long dst = (((long long)b * h_sparse + h) * w + (j % w)) * d + 4 * c4;
  if (sizeof(T) == 4) {
    *reinterpret_cast<float4*>(kc + dst) = *reinterpret_cast<const float4*>(k + src);
    *reinterpret_cast<float4*>(vc + dst) = *reinterpret_cast<const float4*>(v + src);
  } else {
    *reinterpret_cast<uint2*>(kc + dst) = *reinterpret_cast<const uint2*>(k + src);
    *reinterpret_cast<uint2*>(vc + dst) = *reinterpret_cast<const uint2*>(v + src);
  }
}

// ------------------------------------------------------------------------------------
// Decode step: one CTA per (b, h).
// ------------------------------------------------------------------------------------
// A 16-byte load that stays where it is written: two of them in a row are both in flight before the
// first use (left to itself the compiler, short of registers, pairs every load with its use).
__device__ __forceinline__ uint4 ld16_in_order(const void* p) {
  uint4 r;
  asm volatile("ld.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p) : "memory");
  return r;
}
// 16 bytes of a ring row (4 floats or 8 bf16) against the matching entries of a vector in shared memory
template <typename T> struct Row16;
template <> struct Row16<float> {
  static constexpr int kElems = 4;
  static __device__ __forceinline__ float dot(uint4 raw, const float* qv) {
    const float4 q4 = *reinterpret_cast<const float4*>(qv);
    return __uint_as_float(raw.x) * q4.x + __uint_as_float(raw.y) * q4.y + __uint_as_float(raw.z) * q4.z +
           __uint_as_float(raw.w) * q4.w;
  }
  static __device__ __forceinline__ void axpy(uint4 raw, float p, float* acc) {
    acc[0] = fmaf(p, __uint_as_float(raw.x), acc[0]);
    acc[1] = fmaf(p, __uint_as_float(raw.y), acc[1]);
    acc[2] = fmaf(p, __uint_as_float(raw.z), acc[2]);
    acc[3] = fmaf(p, __uint_as_float(raw.w), acc[3]);
  }
};
template <> struct Row16<__nv_bfloat16> {
  static constexpr int kElems = 8;
  static __device__ __forceinline__ float dot(uint4 raw, const float* qv) {
    const float4 qa = *reinterpret_cast<const float4*>(qv), qb = *reinterpret_cast<const float4*>(qv + 4);
    float a0 = __uint_as_float(raw.x << 16) * qa.x, a1 = __uint_as_float(raw.x & 0xffff0000u) * qa.y;
    a0 = fmaf(__uint_as_float(raw.y << 16), qa.z, a0);
    a1 = fmaf(__uint_as_float(raw.y & 0xffff0000u), qa.w, a1);
    a0 = fmaf(__uint_as_float(raw.z << 16), qb.x, a0);
    a1 = fmaf(__uint_as_float(raw.z & 0xffff0000u), qb.y, a1);
    a0 = fmaf(__uint_as_float(raw.w << 16), qb.z, a0);
    a1 = fmaf(__uint_as_float(raw.w & 0xffff0000u), qb.w, a1);
    return a0 + a1;
  }
  static __device__ __forceinline__ void axpy(uint4 raw, float p, float* acc) {
    acc[0] = fmaf(p, __uint_as_float(raw.x << 16), acc[0]);
    acc[1] = fmaf(p, __uint_as_float(raw.x & 0xffff0000u), acc[1]);
    acc[2] = fmaf(p, __uint_as_float(raw.y << 16), acc[2]);
    acc[3] = fmaf(p, __uint_as_float(raw.y & 0xffff0000u), acc[3]);
    acc[4] = fmaf(p, __uint_as_float(raw.z << 16), acc[4]);
    acc[5] = fmaf(p, __uint_as_float(raw.z & 0xffff0000u), acc[5]);
    acc[6] = fmaf(p, __uint_as_float(raw.w << 16), acc[6]);
    acc[7] = fmaf(p, __uint_as_float(raw.w & 0xffff0000u), acc[7]);
  }
};

__device__ __forceinline__ float block_reduce(float x, bool is_max, float* scratch /* 33 floats */) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float y = __shfl_xor_sync(0xffffffffu, x, off);
    x = is_max ? fmaxf(x, y) : x + y;
  }
  __syncthreads();
  if (lane == 0) scratch[wid] = x;
  __syncthreads();
  if (wid == 0) {
    float y = (lane < nw) ? scratch[lane] : (is_max ? -INFINITY : 0.f);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float u = __shfl_xor_sync(0xffffffffu, y, off);
      y = is_max ? fmaxf(y, u) : y + u;
    }
    if (lane == 0) scratch[32] = y;
  }
  __syncthreads();
  return scratch[32];
}

// Seven CTAs per SM: one CTA per (batch, head) then fits a batch of 64 x 16 heads in a single wave.
template <typename T, int D>
__global__ void __launch_bounds__(256, 7)
decode_step_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                   T* __restrict__ o, T* __restrict__ kc, T* __restrict__ vc, float* __restrict__ S,
                   float* __restrict__ z, long long t_all, long long* __restrict__ t_seq, int H, int w,
                   int h_sparse, float scale, const T* __restrict__ W /* [H - h_sparse, D, D] or null: elu + 1 */) {
  constexpr int D4 = D / 4;
  constexpr int G = 256 / D4;  // thread groups along the reduced dimension
  // windowed heads: a ring row is read 16 bytes per thread (a slot's round trip to L2 is what a step
  // waits for, so the fewer rounds the better): TPS threads per slot, GW slots per round
  constexpr int EPT = Row16<T>::kElems, TPS = D / EPT, GW = 256 / TPS;
  extern __shared__ __align__(16) float dyn[];  // window heads: w scores
  __shared__ __align__(16) float qs[D];
  __shared__ __align__(16) float ks[D];
  __shared__ float scratch[33];
  __shared__ __align__(16) float part[GW][D];  // GW >= G

  const int h = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
  const long long io = ((long long)b * H + h) * D;
  const int c4 = tid % D4, grp = tid / D4;
  // Position of this sequence: the whole batch in lock step, or its own entry of t_seq (a negative
  // entry marks an idle slot of the batch: state untouched, output row zero).  The sequence's H
  // CTAs count their arrivals in bits 48..62 of the entry; the last one clears the count and moves
  // the position on, so the step needs no second launch.
  // (A thread that loads none of the step's inputs fetches the position, so that the two global
  // round trips overlap.)
  float qv = 0.f;
  T kin = from_f32<T>(0.f), vin = from_f32<T>(0.f);
  long long t = t_all;
  if (t_seq != nullptr) {
    __shared__ long long t_sh;
    if (tid == 255) {
      long long cur = *reinterpret_cast<const volatile long long*>(t_seq + b);
      if (cur >= 0) {
        unsigned long long* slot = reinterpret_cast<unsigned long long*>(t_seq + b);
        const unsigned long long old = atomicAdd(slot, 1ull << 48);
        cur = (long long)(old & ((1ull << 48) - 1));
        if ((old >> 48) + 1 == (unsigned long long)H) atomicAdd(slot, 1ull - ((unsigned long long)H << 48));
      }
      t_sh = cur;
    }
    if (tid < D) {
      qv = to_f32(q[io + tid]);
      kin = k[io + tid];
      vin = v[io + tid];
    }
    __syncthreads();
    t = t_sh;
  } else if (tid < D) {
    qv = to_f32(q[io + tid]);
    kin = k[io + tid];
    vin = v[io + tid];
  }
  if (t < 0) {
    if (tid < D) o[io + tid] = from_f32<T>(0.f);
    return;
  }

  if (h < h_sparse) {
    T* kcb = kc + ((long long)b * h_sparse + h) * (long long)w * D;
    T* vcb = vc + ((long long)b * h_sparse + h) * (long long)w * D;
    const int cur = (int)(t % w);
    const int nvalid = (t + 1 < (long long)w) ? (int)(t + 1) : w;
    if (tid < D) {
      qs[tid] = qv;
      kcb[(long long)cur * D + tid] = kin;
      vcb[(long long)cur * D + tid] = vin;
    }
    __syncthreads();
    // scores: TPS threads per slot (a warp reads whole cache lines of the ring), partial dot products
    // reduced over the group by shuffles; slot `cur` is read from the step input (same values).  TPS is
    // 8, 16 or 32, so a group never straddles a warp.
    const int cw = tid % TPS, gw = tid / TPS;
    float mloc = -INFINITY;
    for (int s0 = 0; s0 < nvalid; s0 += 2 * GW) {  // uniform trip count: the shuffles below are warp-wide
      const int sa = s0 + gw, sb = s0 + GW + gw;
      uint4 ra = make_uint4(0u, 0u, 0u, 0u), rb = ra;
      if (sa < nvalid) ra = ld16_in_order(((sa == cur) ? (k + io) : (kcb + (long long)sa * D)) + EPT * cw);
      if (sb < nvalid) rb = ld16_in_order(((sb == cur) ? (k + io) : (kcb + (long long)sb * D)) + EPT * cw);
      float acc_a = Row16<T>::dot(ra, &qs[EPT * cw]), acc_b = Row16<T>::dot(rb, &qs[EPT * cw]);
#pragma unroll
      for (int off = TPS / 2; off > 0; off >>= 1) {
        acc_a += __shfl_xor_sync(0xffffffffu, acc_a, off);
        acc_b += __shfl_xor_sync(0xffffffffu, acc_b, off);
      }
      if (cw == 0) {
        if (sa < nvalid) {
          acc_a *= scale;
          dyn[sa] = acc_a;
          mloc = fmaxf(mloc, acc_a);
        }
        if (sb < nvalid) {
          acc_b *= scale;
          dyn[sb] = acc_b;
          mloc = fmaxf(mloc, acc_b);
        }
      }
    }
    const float mx = block_reduce(mloc, true, scratch);
    float lloc = 0.f;
    for (int s = tid; s < nvalid; s += 256) {
      const float p = expf(dyn[s] - mx);
      dyn[s] = p;
      lloc += p;
    }
    const float lsum = block_reduce(lloc, false, scratch);  // barriers inside publish dyn[]
    float accv[EPT];
#pragma unroll
    for (int e = 0; e < EPT; ++e) accv[e] = 0.f;
    for (int sa = gw; sa < nvalid; sa += 2 * GW) {
      const int sb = sa + GW;
      uint4 ra = ld16_in_order(((sa == cur) ? (v + io) : (vcb + (long long)sa * D)) + EPT * cw), rb = make_uint4(0u, 0u, 0u, 0u);
      if (sb < nvalid) rb = ld16_in_order(((sb == cur) ? (v + io) : (vcb + (long long)sb * D)) + EPT * cw);
      Row16<T>::axpy(ra, dyn[sa], accv);
      Row16<T>::axpy(rb, sb < nvalid ? dyn[sb] : 0.f, accv);
    }
#pragma unroll
    for (int e = 0; e < EPT; e += 4)
      *reinterpret_cast<float4*>(&part[gw][EPT * cw + e]) = make_float4(accv[e], accv[e + 1], accv[e + 2], accv[e + 3]);
    __syncthreads();
    if (tid < D) {
      float sum = 0.f;
#pragma unroll
      for (int gi = 0; gi < GW; ++gi) sum += part[gi][tid];
      o[io + tid] = from_f32<T>(sum / lsum);
    }
  } else {
    const long long sidx = (long long)b * (H - h_sparse) + (h - h_sparse);
    float* Sb = S + sidx * D * D;
    float* zb = z + sidx * D;
    float denloc = 0.f;
    if (W != nullptr) {
      // positive random features of q_t and k_t (Sec. III-A / III-C): exp(<w_a, x> - |x|^2 / 2) / sqrt(D)
      // for the key; for the query exp(<w_a, q> - max_a <w_a, q>) (a factor common to its features cancels
      // in the output).  A warp per feature, lanes along the input dimension.
      if (tid < D) {
        part[0][tid] = qv;
        part[1][tid] = to_f32(kin);
      }
      const float n2k = block_reduce(tid < D ? to_f32(kin) * to_f32(kin) : 0.f, false, scratch);  // barriers inside publish part[]
      const T* Wh = W + (long long)(h - h_sparse) * D * D;
      const int lane = tid & 31, wid = tid >> 5;
      for (int a = wid; a < D; a += 8) {
        float pq = 0.f, pk = 0.f;
        for (int cc = lane; cc < D; cc += 32) {
          const float wv = to_f32(Wh[(long long)a * D + cc]);
          pq = fmaf(wv, part[0][cc], pq);
          pk = fmaf(wv, part[1][cc], pk);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
          pq += __shfl_xor_sync(0xffffffffu, pq, off);
          pk += __shfl_xor_sync(0xffffffffu, pk, off);
        }
        if (lane == 0) {
          qs[a] = pq;
          ks[a] = expf(pk - 0.5f * n2k) * rsqrtf((float)D);
        }
      }
      __syncthreads();
      const float pmax = block_reduce(tid < D ? qs[tid] : -INFINITY, true, scratch);
      if (tid < D) qs[tid] = expf(qs[tid] - pmax);
      __syncthreads();
    }
    if (tid < D) {
      const float qp = W != nullptr ? qs[tid] : phi_elu1(qv);
      const float kp = W != nullptr ? ks[tid] : phi_elu1(to_f32(kin));
      qs[tid] = qp;
      ks[tid] = kp;
      const float zn = zb[tid] + kp;
      zb[tid] = zn;
      denloc = qp * zn;
    }
    const float den = block_reduce(denloc, false, scratch);  // barriers inside publish qs/ks
    const float4 vv = Vec4<T>::load(v + io + 4 * c4);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int a = grp; a < D; a += G) {
      float4 s4 = *reinterpret_cast<float4*>(Sb + (long long)a * D + 4 * c4);
      const float kp = ks[a], qp = qs[a];
      s4.x = fmaf(kp, vv.x, s4.x);
      s4.y = fmaf(kp, vv.y, s4.y);
      s4.z = fmaf(kp, vv.z, s4.z);
      s4.w = fmaf(kp, vv.w, s4.w);
      *reinterpret_cast<float4*>(Sb + (long long)a * D + 4 * c4) = s4;
      acc.x = fmaf(qp, s4.x, acc.x);
      acc.y = fmaf(qp, s4.y, acc.y);
      acc.z = fmaf(qp, s4.z, acc.z);
      acc.w = fmaf(qp, s4.w, acc.w);
    }
    *reinterpret_cast<float4*>(&part[grp][4 * c4]) = acc;
    __syncthreads();
    if (tid < D) {
      float sum = 0.f;
#pragma unroll
      for (int gi = 0; gi < G; ++gi) sum += part[gi][tid];
      o[io + tid] = from_f32<T>(sum / den);
    }
  }
}

template <typename T>
cudaError_t window_dispatch(const void* q, const void* k, const void* v, void* o, int B, int N, int d, int w,
                            int fwd, float scale, Strides st, int h_begin, int h_count, cudaStream_t stream) {
  dim3 grid((N + 31) / 32, h_count, B);
  if (d == 64)
    window_simt_kernel<T, 64><<<grid, 128, 0, stream>>>((const T*)q, (const T*)k, (const T*)v, (T*)o, N, w, fwd,
                                                        scale, st, h_begin);
  else
    window_simt_kernel<T, 128><<<grid, 128, 0, stream>>>((const T*)q, (const T*)k, (const T*)v, (T*)o, N, w, fwd,
                                                         scale, st, h_begin);
  note_launch();
  return cudaGetLastError();
}

template <typename T>
cudaError_t linear_dispatch(const void* q, const void* k, const void* v, void* o, int B, int N, int d,
                            Strides st, int h_begin, int h_count, float* S_io, float* z_io, bool zero_init,
                            bool global_sum, cudaStream_t stream, const void* W) {
  dim3 grid(d / 32, h_count, B);
  if (d == 64)
    linear_simt_kernel<T, 64><<<grid, 256, 0, stream>>>((const T*)q, (const T*)k, (const T*)v, (T*)o, N, st, h_begin,
                                                        h_count, S_io, z_io, zero_init ? 1 : 0, global_sum ? 1 : 0,
                                                        (const T*)W);
  else
    linear_simt_kernel<T, 128><<<grid, 256, 0, stream>>>((const T*)q, (const T*)k, (const T*)v, (T*)o, N, st, h_begin,
                                                         h_count, S_io, z_io, zero_init ? 1 : 0, global_sum ? 1 : 0,
                                                         (const T*)W);
  note_launch();
  return cudaGetLastError();
}

template <typename T>
cudaError_t decode_dispatch(const void* q, const void* k, const void* v, void* o, void* kc, void* vc, float* S,
                            float* z, long long t, long long* t_seq, int B, int H, int d, int w, int h_sparse,
                            float scale, cudaStream_t stream, const void* W) {
  dim3 grid(H, B);
  const size_t dyn = (size_t)w * sizeof(float);
  if (d == 64) {
    auto kern = decode_step_kernel<T, 64>;
    if (dyn > 40 * 1024) {
      cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
      if (e != cudaSuccess) return e;
    }
    kern<<<grid, 256, dyn, stream>>>((const T*)q, (const T*)k, (const T*)v, (T*)o, (T*)kc, (T*)vc, S, z, t, t_seq,
                                     H, w, h_sparse, scale, (const T*)W);
  } else {
    auto kern = decode_step_kernel<T, 128>;
    if (dyn > 40 * 1024) {
      cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
      if (e != cudaSuccess) return e;
    }
    kern<<<grid, 256, dyn, stream>>>((const T*)q, (const T*)k, (const T*)v, (T*)o, (T*)kc, (T*)vc, S, z, t, t_seq,
                                     H, w, h_sparse, scale, (const T*)W);
  }
  note_launch();
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_window_simt(const void* q, const void* k, const void* v, void* o, int B, int N, int d, int w,
                               int fwd, float scale, int dtype, Strides st, int h_begin, int h_count,
                               cudaStream_t stream) {
  if (h_count <= 0 || B <= 0) return cudaSuccess;
  if (dtype == GF_F32)
    return window_dispatch<float>(q, k, v, o, B, N, d, w, fwd, scale, st, h_begin, h_count, stream);
  return window_dispatch<__nv_bfloat16>(q, k, v, o, B, N, d, w, fwd, scale, st, h_begin, h_count, stream);
}

cudaError_t launch_linear_simt(const void* q, const void* k, const void* v, void* o, int B, int N, int d,
                               int dtype, Strides st, int h_begin, int h_count, float* S_io, float* z_io,
                               bool zero_init, cudaStream_t stream, bool global_sum, const void* W) {
  if (h_count <= 0 || B <= 0) return cudaSuccess;
  if (dtype == GF_F32)
    return linear_dispatch<float>(q, k, v, o, B, N, d, st, h_begin, h_count, S_io, z_io, zero_init, global_sum,
                                  stream, W);
  return linear_dispatch<__nv_bfloat16>(q, k, v, o, B, N, d, st, h_begin, h_count, S_io, z_io, zero_init, global_sum,
                                        stream, W);
}

cudaError_t launch_export_ring(const void* k, const void* v, void* k_cache, void* v_cache, int B, int N, int d,
                               int w, int dtype, Strides st, int h_sparse, cudaStream_t stream) {
  if (h_sparse <= 0 || B <= 0) return cudaSuccess;
  const int wn = N < w ? N : w;
  const long long total4 = (long long)B * h_sparse * wn * (d / 4);
  const int threads = 256;
  const long long blocks = (total4 + threads - 1) / threads;
  if (dtype == GF_F32)
    export_ring_kernel<float><<<(unsigned)blocks, threads, 0, stream>>>(
        (const float*)k, (const float*)v, (float*)k_cache, (float*)v_cache, N, d, w, wn, st, h_sparse, total4);
  else
    export_ring_kernel<__nv_bfloat16><<<(unsigned)blocks, threads, 0, stream>>>(
        (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (__nv_bfloat16*)k_cache, (__nv_bfloat16*)v_cache, N,
        d, w, wn, st, h_sparse, total4);
  note_launch();
  return cudaGetLastError();
}

namespace {
__global__ void wait_placed_kernel(const unsigned int* placed, unsigned int target, unsigned int max_ns) {
  unsigned long long t0, t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
  for (int i = 0; i < 100000; ++i) {  // bounded whatever the timer does
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(placed) : "memory");
    if (v >= target) break;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    if (t - t0 >= max_ns) break;
    __nanosleep(100);
  }
}
}  // namespace

__global__ void set_header_kernel(WsHeader* ws, unsigned int wait_kcycles, unsigned int drop_flag) {
  ws->wait_kcycles = wait_kcycles;
  ws->drop_flag = drop_flag;
}

cudaError_t launch_set_header(WsHeader* ws, unsigned int wait_kcycles, unsigned int drop_flag, cudaStream_t stream) {
  set_header_kernel<<<1, 1, 0, stream>>>(ws, wait_kcycles, drop_flag);
  note_launch();
  return cudaGetLastError();
}

cudaError_t launch_wait_placed(WsHeader* ws, unsigned int target, unsigned int max_ns, cudaStream_t stream) {
  wait_placed_kernel<<<1, 1, 0, stream>>>(&ws->placed, target, max_ns);
  note_launch();
  return cudaGetLastError();
}

cudaError_t launch_decode_step(const void* q, const void* k, const void* v, void* o, void* k_cache,
                               void* v_cache, float* S, float* z, long long t, long long* t_seq, int B, int H,
                               int d, int w, int h_sparse, float scale, int dtype, cudaStream_t stream,
                               const void* W) {
  if (dtype == GF_F32)
    return decode_dispatch<float>(q, k, v, o, k_cache, v_cache, S, z, t, t_seq, B, H, d, w, h_sparse, scale,
                                  stream, W);
  return decode_dispatch<__nv_bfloat16>(q, k, v, o, k_cache, v_cache, S, z, t, t_seq, B, H, d, w, h_sparse, scale,
                                        stream, W);
}

}  // namespace gf
