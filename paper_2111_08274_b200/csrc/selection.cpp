#include "selection.h"

#include <math.h>

#include "philox.cuh"

namespace hadfl {

double quartile3(const double *x, int n) {
  double s[64];
  for (int i = 0; i < n; ++i) {  // insertion sort: n <= 32
    double v = x[i];
    int j = i;
    while (j > 0 && s[j - 1] > v) {
      s[j] = s[j - 1];
      --j;
    }
    s[j] = v;
  }
  const double h = 0.75 * (double)(n - 1);
  const int lo = (int)h;
  if (lo + 1 >= n) return s[n - 1];
  return s[lo] + (h - (double)lo) * (s[lo + 1] - s[lo]);
}

int selection_weights(const double *x, const uint8_t *avail, int n, double *wgt) {
  double xs[64];
  int n_avail = 0;
  for (int i = 0; i < n; ++i)
    if (!avail || avail[i]) xs[n_avail++] = x[i];
  for (int i = 0; i < n; ++i) wgt[i] = 0.0;
  if (n_avail == 0) return 0;
  const double mu = quartile3(xs, n_avail);
  double l[64];
  double lmax = -INFINITY;
  for (int i = 0; i < n; ++i) {
    if (avail && !avail[i]) continue;
    const double d = x[i] - mu;
    l[i] = -(d * d) / 2.0;
    lmax = l[i] > lmax ? l[i] : lmax;
  }
  for (int i = 0; i < n; ++i)
    if (!avail || avail[i]) wgt[i] = exp(l[i] - lmax);
  return n_avail;
}

bool selection_probs(const double *x, const uint8_t *avail, int n, double *P) {
  double wgt[64];
  if (selection_weights(x, avail, n, wgt) == 0) return false;
  double W = 0.0;
  for (int i = 0; i < n; ++i)
    if (!avail || avail[i]) W += wgt[i];
  for (int i = 0; i < n; ++i) P[i] = (!avail || avail[i]) ? wgt[i] / W : 0.0;
  return true;
}

static uint64_t draw_bits(const PhiloxKeys &keys, int64_t round, uint32_t t) {
  const uint64_t r = (uint64_t)round;
  uint32_t c0 = t, c1 = 0u, c2 = (uint32_t)r, c3 = kTagSelect | ((uint32_t)(r >> 32) & 0xFFFFFFu);
  philox4x32_10(c0, c1, c2, c3, keys);
  return ((uint64_t)c1 << 32) | c0;
}

bool selection_draw(const double *x, const uint8_t *avail, int n, int64_t round, uint64_t seed,
                    int k, int32_t *out) {
  double wgt[64];
  const int n_avail = selection_weights(x, avail, n, wgt);
  if (k < 1 || k > n_avail) return false;
  const PhiloxKeys keys = expand_keys(seed);
  bool in_pool[64];
  for (int i = 0; i < n; ++i) in_pool[i] = !avail || avail[i];
  int pool = n_avail;
  for (int t = 0; t < k; ++t, --pool) {
    const uint64_t bits = draw_bits(keys, round, (uint32_t)t);
    double W = 0.0;
    for (int i = 0; i < n; ++i)
      if (in_pool[i]) W += wgt[i];
    int pick = -1;
    if (W > 0.0) {
      const double target = ((double)(bits >> 11) * 0x1p-53) * W;
      double c = 0.0;
      int fallback = -1;
      for (int i = 0; i < n && pick < 0; ++i) {
        if (!in_pool[i]) continue;
        if (wgt[i] > 0.0) fallback = i;
        c += wgt[i];
        if (c > target) pick = i;
      }
      if (pick < 0) pick = fallback;
    } else {
      // all remaining weights underflowed: stragglers still get their turn, uniformly
      int skip = (int)(bits % (uint64_t)pool);
      for (int i = 0; i < n; ++i) {
        if (!in_pool[i]) continue;
        if (skip-- == 0) {
          pick = i;
          break;
        }
      }
    }
    in_pool[pick] = false;
    out[t] = pick;
  }
  return true;
}

void aggregation_weights(int mode, const double *x, const uint8_t *avail, int n,
                         const int32_t *sel, int k, float *a) {
  if (mode == 0 || k == 1) {
    const float u = (float)(1.0 / (double)k);
    for (int j = 0; j < k; ++j) a[j] = u;
    return;
  }
  double xs[64];
  int n_avail = 0;
  for (int i = 0; i < n; ++i)
    if (!avail || avail[i]) xs[n_avail++] = x[i];
  const double mu = quartile3(xs, n_avail);
  double l[64], lmax = -INFINITY;
  for (int j = 0; j < k; ++j) {
    const double d = x[sel[j]] - mu;
    l[j] = -(d * d) / 2.0;
    lmax = l[j] > lmax ? l[j] : lmax;
  }
  double b[64], B = 0.0;
  for (int j = 0; j < k; ++j) {
    b[j] = exp(l[j] - lmax);
    B += b[j];
  }
  float head = 0.f;
  for (int j = 0; j + 1 < k; ++j) {
    a[j] = (float)(b[j] / B);
    head += a[j];
  }
  a[k - 1] = 1.0f - head;
}

double predict_version(const double *series, int n_obs, double alpha, double m) {
  double s1 = series[0], s2 = series[0];
  for (int j = 1; j < n_obs; ++j) {
    s1 = alpha * series[j] + (1.0 - alpha) * s1;
    s2 = alpha * s1 + (1.0 - alpha) * s2;
  }
  return (2.0 * s1 - s2) + alpha / (1.0 - alpha) * (s1 - s2) * m;
}

}  // namespace hadfl
