/*
 * GFormer hybrid attention -- plain fp64 CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, literal statement of what the
 * hybrid attention layer computes.  It shares no code with the CUDA library and
 * the CUDA library never calls it; only the tests, the smoke check and the CPU
 * baseline leg of the benchmark may load it.
 *
 * Everything is fp64.  Tensors are dense row-major [B, H, N, d] (one head of one
 * batch element is a contiguous N x d block); indices are 0-based.
 *
 * What each function follows in the paper:
 *   window head   Eq. 1 (softmax(Q K^T / sqrt(D)) V), the causal mask of Sec. II-A
 *                 (masked logits are -inf, i.e. they drop out of the sums) and the
 *                 fixed left window of Sec. III-B.  Reading taken: the window of
 *                 token i is the w keys j in [i-w+1, i] (itself plus the w-1 tokens
 *                 before it), truncated at the sequence start.
 *   linear head   Algorithm 1 (causal linear attention): running A += phi(K_i) (x) V_i,
 *                 Z += phi(K_i), readout H_i = phi(Q_i)^T A / (phi(Q_i) . Z) taken
 *                 AFTER the two updates of step i (inclusive prefix).  The readout
 *                 line is garbled in print; this is the repaired reading.
 *   phi           Sec. II-B: phi(x) = elu(x) + 1 (element by element).
 *   phi_W         Sec. III-A / III-C name "positive orthogonal random features" as the feature map of
 *                 the linear heads without printing a formula; the formula is the cited Performer
 *                 paper's positive random feature map of the softmax kernel,
 *                     phi_W(x)[a] = exp(<w_a, x> - |x|^2 / 2) / sqrt(m),   a = 0 .. m-1,
 *                 with a caller-supplied projection W = (w_a) per head.  m = d, because the state of
 *                 Algorithm 1 is E x E.  No stabiliser is subtracted and no extra scale is applied
 *                 to x (the linear heads carry no 1/sqrt(D), reading P3): what the caller passes
 *                 is what is projected.  Whether the rows of W are orthogonal is the caller's
 *                 business (a property of the input, generated outside this file).
 *   hybrid        Sec. III-A: heads are split along H; the first h_sparse heads are
 *                 windowed, the rest linear; every head writes its own slot of O.
 *   decode        Algorithm 1 advanced one token at a time plus the window rule on a
 *                 ring buffer of w cached keys/values (token j lives in slot j mod w).
 *   "self" layer  (the bidirectional variant of Sec. II-A used for ViT, Sec. IV-D/E)
 *                 window head: Eq. 1 without the
 *                 causal mask, over a two-sided window.  The paper does not print the
 *                 two-sided rule; reading taken: token i sees the keys j with |i - j| < w
 *                 (itself, the w-1 tokens before and the w-1 after), truncated at both
 *                 ends -- the causal window mirrored.  Linear head: the unmasked form of
 *                 Sec. II-B, phi(Q) (phi(K)^T V), every row normalised like Algorithm 1
 *                 does, by phi(Q_i) . sum_j phi(K_j) over all j.
 *
 * No blocking, no fusion, no reordering: loops are in the paper's order.
 * OpenMP is used only across independent (batch, head) pairs.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int gfo_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Sec. II-B: phi(x) = elu(x) + 1  ( = x + 1 for x > 0, exp(x) otherwise ). */
double gfo_phi(double x) { return x > 0.0 ? x + 1.0 : exp(x); }

void gfo_phi_array(const double* x, double* y, long n) {
  for (long i = 0; i < n; ++i) y[i] = gfo_phi(x[i]);
}

/* The positive random feature map of one vector: out[a] = exp(<W[a], x> - |x|^2 / 2) / sqrt(d),
 * W is d x d row-major (row a = projection vector w_a). */
void gfo_phi_favor(const double* x, const double* W, int d, double* out) {
  double n2 = 0.0;
  for (int c = 0; c < d; ++c) n2 += x[c] * x[c];
  for (int a = 0; a < d; ++a) {
    double proj = 0.0;
    for (int c = 0; c < d; ++c) proj += W[(size_t)a * d + c] * x[c];
    out[a] = exp(proj - 0.5 * n2) / sqrt((double)d);
  }
}

/* Feature map of the linear heads: elu + 1 element by element (W == NULL), or phi_W. */
static void feature_map(const double* x, const double* W, int d, double* out) {
  if (W) gfo_phi_favor(x, W, d, out);
  else for (int a = 0; a < d; ++a) out[a] = gfo_phi(x[a]);
}

/* One windowed head: q, k, v, o are N x d. */
static void window_head(const double* q, const double* k, const double* v, double* o,
                        long N, int d, long w, double scale, double* e /* >= min(w,N) */) {
  for (long i = 0; i < N; ++i) {
    long lo = i - w + 1;
    if (lo < 0) lo = 0;
    /* logits of the window (Eq. 1 restricted to the unmasked band) */
    double m = -INFINITY;
    for (long j = lo; j <= i; ++j) {
      double s = 0.0;
      for (int c = 0; c < d; ++c) s += q[i * d + c] * k[j * d + c];
      s *= scale;
      e[j - lo] = s;
      if (s > m) m = s;
    }
    /* softmax over the window */
    double l = 0.0;
    for (long j = lo; j <= i; ++j) {
      e[j - lo] = exp(e[j - lo] - m);
      l += e[j - lo];
    }
    /* weighted sum of values */
    for (int c = 0; c < d; ++c) {
      double acc = 0.0;
      for (long j = lo; j <= i; ++j) acc += e[j - lo] * v[j * d + c];
      o[i * d + c] = acc / l;
    }
  }
}

/* One linear head, Algorithm 1.  S is d x d (S[a*d + c], a = feature index of
 * phi(k), c = value index), z is d.  Both are read as the initial state and left
 * holding the final state. */
static void linear_head(const double* q, const double* k, const double* v, double* o,
                        long N, int d, double* S, double* z, double* qp, double* kp, const double* W) {
  for (long i = 0; i < N; ++i) {
    feature_map(q + i * d, W, d, qp);
    feature_map(k + i * d, W, d, kp);
    for (int a = 0; a < d; ++a) {
      for (int c = 0; c < d; ++c) S[a * d + c] += kp[a] * v[i * d + c];
      z[a] += kp[a];
    }
    double den = 0.0;
    for (int a = 0; a < d; ++a) den += qp[a] * z[a];
    for (int c = 0; c < d; ++c) {
      double num = 0.0;
      for (int a = 0; a < d; ++a) num += qp[a] * S[a * d + c];
      o[i * d + c] = num / den;
    }
  }
}

/* One two-sided windowed head ("self" variant): keys j with |i - j| < w. */
static void window_head_sym(const double* q, const double* k, const double* v, double* o,
                            long N, int d, long w, double scale, double* e /* >= min(2w-1,N) */) {
  for (long i = 0; i < N; ++i) {
    long lo = i - w + 1, hi = i + w - 1;
    if (lo < 0) lo = 0;
    if (hi > N - 1) hi = N - 1;
    double m = -INFINITY;
    for (long j = lo; j <= hi; ++j) {
      double s = 0.0;
      for (int c = 0; c < d; ++c) s += q[i * d + c] * k[j * d + c];
      s *= scale;
      e[j - lo] = s;
      if (s > m) m = s;
    }
    double l = 0.0;
    for (long j = lo; j <= hi; ++j) {
      e[j - lo] = exp(e[j - lo] - m);
      l += e[j - lo];
    }
    for (int c = 0; c < d; ++c) {
      double acc = 0.0;
      for (long j = lo; j <= hi; ++j) acc += e[j - lo] * v[j * d + c];
      o[i * d + c] = acc / l;
    }
  }
}

/* One global (unmasked) linear head, Sec. II-B: S = sum_j phi(K_j) (x) V_j and z = sum_j
 * phi(K_j) over the whole sequence first, then H_i = phi(Q_i)^T S / (phi(Q_i) . z). */
static void linear_head_global(const double* q, const double* k, const double* v, double* o,
                               long N, int d, double* S, double* z, double* qp, const double* W) {
  memset(S, 0, sizeof(double) * (size_t)d * (size_t)d);
  memset(z, 0, sizeof(double) * (size_t)d);
  for (long j = 0; j < N; ++j) {
    feature_map(k + j * d, W, d, qp);
    for (int a = 0; a < d; ++a) {
      for (int c = 0; c < d; ++c) S[a * d + c] += qp[a] * v[j * d + c];
      z[a] += qp[a];
    }
  }
  for (long i = 0; i < N; ++i) {
    double den = 0.0;
    feature_map(q + i * d, W, d, qp);
    for (int a = 0; a < d; ++a) den += qp[a] * z[a];
    for (int c = 0; c < d; ++c) {
      double num = 0.0;
      for (int a = 0; a < d; ++a) num += qp[a] * S[a * d + c];
      o[i * d + c] = num / den;
    }
  }
}

/* The "self" hybrid layer: heads [0, h_sparse) two-sided windowed, heads [h_sparse, H) global
 * linear (Sec. III-A routing, unchanged). */
void gfo_hybrid_attn_self(const double* q, const double* k, const double* v, double* o,
                          long B, long H, long N, int d, long w, long h_sparse, double scale,
                          const double* W /* [H - h_sparse, d, d] or NULL: elu + 1 */) {
  long span = 2 * w - 1 < N ? 2 * w - 1 : N;
#pragma omp parallel
  {
    double* e = (double*)malloc(sizeof(double) * (size_t)(span > 0 ? span : 1));
    double* S = (double*)malloc(sizeof(double) * ((size_t)d * (size_t)d + 2 * (size_t)d));
#pragma omp for schedule(dynamic, 1)
    for (long bh = 0; bh < B * H; ++bh) {
      size_t off = (size_t)bh * (size_t)N * (size_t)d;
      if (bh % H < h_sparse) window_head_sym(q + off, k + off, v + off, o + off, N, d, w, scale, e);
      else linear_head_global(q + off, k + off, v + off, o + off, N, d, S, S + (size_t)d * d, S + (size_t)d * d + d,
                              W ? W + (size_t)(bh % H - h_sparse) * d * d : NULL);
    }
    free(e);
    free(S);
  }
}

/* Windowed softmax attention on all B*H heads. */
void gfo_window_attn(const double* q, const double* k, const double* v, double* o,
                     long B, long H, long N, int d, long w, double scale) {
  long wn = w < N ? w : N;
#pragma omp parallel
  {
    double* e = (double*)malloc(sizeof(double) * (size_t)(wn > 0 ? wn : 1));
#pragma omp for schedule(dynamic, 1)
    for (long bh = 0; bh < B * H; ++bh) {
      size_t off = (size_t)bh * (size_t)N * (size_t)d;
      window_head(q + off, k + off, v + off, o + off, N, d, w, scale, e);
    }
    free(e);
  }
}

/* Causal linear attention on all B*H heads.  S_io [B,H,d,d] and z_io [B,H,d] may be
 * NULL (fresh zero state, final state discarded). */
void gfo_causal_linear_attn(const double* q, const double* k, const double* v, double* o,
                            long B, long H, long N, int d, double* S_io, double* z_io,
                            const double* W /* [H, d, d] or NULL: elu + 1 */) {
#pragma omp parallel
  {
    double* S = (double*)malloc(sizeof(double) * (size_t)d * (size_t)d);
    double* z = (double*)malloc(sizeof(double) * (size_t)d * 3);
#pragma omp for schedule(dynamic, 1)
    for (long bh = 0; bh < B * H; ++bh) {
      size_t off = (size_t)bh * (size_t)N * (size_t)d;
      if (S_io) memcpy(S, S_io + (size_t)bh * d * d, sizeof(double) * (size_t)d * d);
      else memset(S, 0, sizeof(double) * (size_t)d * d);
      if (z_io) memcpy(z, z_io + (size_t)bh * d, sizeof(double) * (size_t)d);
      else memset(z, 0, sizeof(double) * (size_t)d);
      linear_head(q + off, k + off, v + off, o + off, N, d, S, z, z + d, z + 2 * d,
                  W ? W + (size_t)(bh % H) * d * d : NULL);
      if (S_io) memcpy(S_io + (size_t)bh * d * d, S, sizeof(double) * (size_t)d * d);
      if (z_io) memcpy(z_io + (size_t)bh * d, z, sizeof(double) * (size_t)d);
    }
    free(S);
    free(z);
  }
}

/* Hybrid layer: heads [0, h_sparse) windowed, heads [h_sparse, H) linear.
 * Optional state export for decoding (any of them may be NULL):
 *   k_cache, v_cache [B, h_sparse, w, d]: the last min(N, w) keys/values of the
 *       windowed heads, token j in slot j mod w (other slots untouched);
 *   S_out [B, H - h_sparse, d, d], z_out [B, H - h_sparse, d]: final linear state. */
void gfo_hybrid_attn(const double* q, const double* k, const double* v, double* o,
                     long B, long H, long N, int d, long w, long h_sparse, double scale,
                     double* k_cache, double* v_cache, double* S_out, double* z_out,
                     const double* W /* [H - h_sparse, d, d] or NULL: elu + 1 */) {
  long H1 = H - h_sparse;
  long wn = w < N ? w : N;
#pragma omp parallel
  {
    double* e = (double*)malloc(sizeof(double) * (size_t)(wn > 0 ? wn : 1));
    double* S = (double*)malloc(sizeof(double) * (size_t)d * (size_t)d);
    double* z = (double*)malloc(sizeof(double) * (size_t)d * 3);
#pragma omp for schedule(dynamic, 1)
    for (long bh = 0; bh < B * H; ++bh) {
      long b = bh / H, h = bh % H;
      size_t off = (size_t)bh * (size_t)N * (size_t)d;
      if (h < h_sparse) {
        window_head(q + off, k + off, v + off, o + off, N, d, w, scale, e);
        if (k_cache && v_cache) {
          size_t coff = ((size_t)b * h_sparse + h) * (size_t)w * d;
          long first = N - wn;
          for (long j = first; j < N; ++j) {
            memcpy(k_cache + coff + (size_t)(j % w) * d, k + off + (size_t)j * d, sizeof(double) * d);
            memcpy(v_cache + coff + (size_t)(j % w) * d, v + off + (size_t)j * d, sizeof(double) * d);
          }
        }
      } else {
        memset(S, 0, sizeof(double) * (size_t)d * d);
        memset(z, 0, sizeof(double) * (size_t)d);
        linear_head(q + off, k + off, v + off, o + off, N, d, S, z, z + d, z + 2 * d,
                    W ? W + (size_t)(h - h_sparse) * d * d : NULL);
        size_t soff = (size_t)b * H1 + (h - h_sparse);
        if (S_out) memcpy(S_out + soff * d * d, S, sizeof(double) * (size_t)d * d);
        if (z_out) memcpy(z_out + soff * d, z, sizeof(double) * (size_t)d);
      }
    }
    free(e);
    free(S);
    free(z);
  }
}

/* One decoding step for token index t (t tokens have been absorbed before it).
 * q, k, v, o are [B, H, d].  Windowed heads: write k, v into ring slot t mod w, then
 * softmax over the min(t+1, w) valid slots.  Linear heads: one iteration of
 * Algorithm 1 on the carried (S, z). */
void gfo_decode_step(const double* q, const double* k, const double* v, double* o,
                     double* k_cache, double* v_cache, double* S, double* z, long t,
                     long B, long H, int d, long w, long h_sparse, double scale,
                     const double* W /* [H - h_sparse, d, d] or NULL: elu + 1 */) {
  long H1 = H - h_sparse;
#pragma omp parallel
  {
    double* e = (double*)malloc(sizeof(double) * (size_t)(w > 0 ? w : 1));
    double* qp = (double*)malloc(sizeof(double) * (size_t)d * 2);
#pragma omp for schedule(dynamic, 1)
    for (long bh = 0; bh < B * H; ++bh) {
      long b = bh / H, h = bh % H;
      const double* qi = q + (size_t)bh * d;
      const double* ki = k + (size_t)bh * d;
      const double* vi = v + (size_t)bh * d;
      double* oi = o + (size_t)bh * d;
      if (h < h_sparse) {
        double* kc = k_cache + ((size_t)b * h_sparse + h) * (size_t)w * d;
        double* vc = v_cache + ((size_t)b * h_sparse + h) * (size_t)w * d;
        memcpy(kc + (size_t)(t % w) * d, ki, sizeof(double) * d);
        memcpy(vc + (size_t)(t % w) * d, vi, sizeof(double) * d);
        long lo = t - w + 1;
        if (lo < 0) lo = 0;
        double m = -INFINITY;
        for (long j = lo; j <= t; ++j) {
          const double* kj = kc + (size_t)(j % w) * d;
          double s = 0.0;
          for (int c = 0; c < d; ++c) s += qi[c] * kj[c];
          s *= scale;
          e[j - lo] = s;
          if (s > m) m = s;
        }
        double l = 0.0;
        for (long j = lo; j <= t; ++j) {
          e[j - lo] = exp(e[j - lo] - m);
          l += e[j - lo];
        }
        for (int c = 0; c < d; ++c) {
          double acc = 0.0;
          for (long j = lo; j <= t; ++j) acc += e[j - lo] * vc[(size_t)(j % w) * d + c];
          oi[c] = acc / l;
        }
      } else {
        size_t soff = (size_t)b * H1 + (h - h_sparse);
        linear_head(qi, ki, vi, oi, 1, d, S + soff * d * d, z + soff * d, qp, qp + d,
                    W ? W + (size_t)(h - h_sparse) * d * d : NULL);
      }
    }
    free(e);
    free(qp);
  }
}
