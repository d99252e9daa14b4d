// Host-side planning arithmetic of the coordinator's strategy generator: the probability-based
// selection function (Eq. 8), the version-dependent aggregation weights built from the same
// function, and the runtime version predictor (Eq. 7).  N <= 32 scalars per call, double
// precision, no GPU involvement.
#pragma once
#include <stdint.h>

namespace hadfl {

// Third quartile of n values by linear interpolation between order statistics.
double quartile3(const double *x, int n);

// Relative selection weights exp(-(x_i - mu)^2 / 2) / max (0 for unavailable devices).
// Returns the number of available devices.
int selection_weights(const double *x, const uint8_t *avail, int n, double *wgt);

// Eq. 8: P(i) = f(x_i) / sum f.  Returns false if no device is available.
bool selection_probs(const double *x, const uint8_t *avail, int n, double *P);

// k sequential weighted draws without replacement; false if k is out of range.
bool selection_draw(const double *x, const uint8_t *avail, int n, int64_t round, uint64_t seed,
                    int k, int32_t *out);

// Aggregation weights a_j for the selected devices.
void aggregation_weights(int mode, const double *x, const uint8_t *avail, int n,
                         const int32_t *sel, int k, float *a);

// Eq. 7.
double predict_version(const double *series, int n_obs, double alpha, double m);

}  // namespace hadfl
