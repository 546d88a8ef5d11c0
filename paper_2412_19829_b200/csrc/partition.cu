// Head partition between the sparse (windowed) and the linear heads: Algorithm 2 and the FLOP
// model of Sec. III-D.  Host arithmetic only (fp64); no device work, no allocation.
#include <math.h>

#include "gformer.h"

namespace {

bool positive_finite(double x) { return x > 0.0 && isfinite(x); }

}  // namespace

extern "C" {

// Algorithm 2: latency0 = p size flops_per0 / perf0 and latency1 = (1 - p) size flops_per1 / perf1
// are both linear in p, so they meet at p' = c1 / (c0 + c1) with c_i = flops_per_i / perf_i
// (size cancels).
int gformer_partition_balance(double flops_per0, double flops_per1, double perf0, double perf1, double* p_out) {
  if (p_out == nullptr) return GF_ERR_INVALID_ARG;
  if (!positive_finite(flops_per0) || !positive_finite(flops_per1) || !positive_finite(perf0) ||
      !positive_finite(perf1))
    return GF_ERR_INVALID_ARG;
  const double c0 = flops_per0 / perf0, c1 = flops_per1 / perf1;
  if (!positive_finite(c0) || !positive_finite(c1) || !positive_finite(c0 + c1)) return GF_ERR_INVALID_ARG;
  *p_out = c1 / (c0 + c1);
  return GF_OK;
}

// FLOP model of Sec. III-D: linear heads 8 B N (H1 E)^2 / perf_linear, sparse heads
// 5 B H0 N W / perf_sparse, H0 + H1 = H.  With x = H1 the two meet where a x^2 + b x - b H = 0,
// a = 8 E^2 / perf_linear, b = 5 W / perf_sparse (B N cancels); the positive root, written so that
// nothing cancels, is x = 2 b H / (b + sqrt(b^2 + 4 a b H)).  sparse - linear grows with H0, so
// the whole number of heads with the smallest gap is one of the two next to H - x.
int gformer_partition_heads(int B, int H, int N, int E, int W, double perf_sparse, double perf_linear,
                            int* h_sparse_out, double* latency_sparse_out, double* latency_linear_out) {
  if (h_sparse_out == nullptr) return GF_ERR_INVALID_ARG;
  if (B < 1 || H < 1 || N < 1 || E < 1 || W < 1) return GF_ERR_INVALID_ARG;
  if (!positive_finite(perf_sparse) || !positive_finite(perf_linear)) return GF_ERR_INVALID_ARG;
  const double bn = (double)B * (double)N;
  auto sparse = [&](int h0) { return 5.0 * bn * (double)h0 * (double)W / perf_sparse; };
  auto linear = [&](int h0) {
    const double he = (double)(H - h0) * (double)E;
    return 8.0 * bn * he * he / perf_linear;
  };
  const double a = 8.0 * (double)E * (double)E / perf_linear, b = 5.0 * (double)W / perf_sparse;
  const double x = 2.0 * b * (double)H / (b + sqrt(b * b + 4.0 * a * b * (double)H));
  if (!isfinite(x)) return GF_ERR_INVALID_ARG;
  int lo = (int)floor((double)H - x) - 1;
  if (lo < 0) lo = 0;
  int hi = lo + 3;
  if (hi > H) hi = H;
  int best = lo;
  double best_gap = fabs(sparse(lo) - linear(lo));
  for (int h0 = lo + 1; h0 <= hi; ++h0) {
    const double gap = fabs(sparse(h0) - linear(h0));
    if (gap < best_gap) { best_gap = gap; best = h0; }
  }
  *h_sparse_out = best;
  if (latency_sparse_out) *latency_sparse_out = sparse(best);
  if (latency_linear_out) *latency_linear_out = linear(best);
  return GF_OK;
}

// What the two micro-benchmarks say in the section's own units.  One windowed head alone costs
// 5 B N W / perf_sparse under the model, and H linear heads together 8 B N (H E)^2 / perf_linear
// (the printed formula is quadratic in the head count), so the rates are those expressions over
// the measured times; the balanced head count rounds p' H to the nearest whole number.
int gformer_partition_from_times(int B, int H, int N, int E, int W, double seconds_per_sparse_head,
                                 double seconds_per_linear_head, double* p_out, int* h_sparse_out,
                                 double* perf_sparse_out, double* perf_linear_out) {
  if (p_out == nullptr || h_sparse_out == nullptr || perf_sparse_out == nullptr || perf_linear_out == nullptr)
    return GF_ERR_INVALID_ARG;
  if (B < 1 || H < 1 || N < 1 || E < 1 || W < 1) return GF_ERR_INVALID_ARG;
  if (!positive_finite(seconds_per_sparse_head) || !positive_finite(seconds_per_linear_head)) return GF_ERR_INVALID_ARG;
  double p = 0.0;
  const int rc = gformer_partition_balance(seconds_per_sparse_head, seconds_per_linear_head, 1.0, 1.0, &p);
  if (rc != GF_OK) return rc;
  int h0 = (int)floor(p * (double)H + 0.5);
  if (h0 < 0) h0 = 0;
  if (h0 > H) h0 = H;
  const double bn = (double)B * (double)N, he = (double)H * (double)E;
  *p_out = p;
  *h_sparse_out = h0;
  *perf_sparse_out = 5.0 * bn * (double)W / seconds_per_sparse_head;
  *perf_linear_out = 8.0 * bn * he * he / ((double)H * seconds_per_linear_head);
  return GF_OK;
}

}  // extern "C"
