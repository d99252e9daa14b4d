// CPU oracle for the HADFL round hot path (Cao et al., "HADFL: Heterogeneity-aware
// Decentralized Federated Learning Framework", arXiv 2111.08274).
//
// THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, single-threaded restatement of what one
// training round computes, written so that a reader can check it against the paper by eye.
// It shares no code, header, table or constant generator with the CUDA library, is never
// called by the product path, and exists only so that tests, the smoke check and the
// benchmark's CPU-baseline leg have something independent to compare against and to time.
//
// What each function follows:
//   * local update            - Eq. 3 (local SGD step) and Algorithm 1 (E_k steps per device),
//                               extended with momentum / weight decay in the PyTorch-SGD
//                               convention (the paper's Eq. 3 is the momentum=0, wd=0 case).
//   * partial aggregation     - Eq. 5: mean of the replicas whose Flag is 1 (K read as the
//                               number of selected devices), written back to those replicas.
//   * global synchronisation  - Algorithm 1 "send w to devices whose Flag = 0": overwrite.
//   * selection               - Eq. 8: P(i) = f(v_i) / sum_n f(v_n) over the available devices,
//                               f the unit-variance Gaussian density about mu, mu the third
//                               quartile of the versions; N_p devices are then drawn one after
//                               the other without replacement; the draw order is the ring order.
//   * version prediction      - Eq. 7 (Brown's double exponential smoothing).
//   * integration             - Section "Model aggregation and fault-tolerant": an unselected device
//                               mixes the received model into its own (a reading offered beside the
//                               overwrite of Algorithm 1; the paper gives no formula).
//   * reduced-precision state - not in the paper: parameters (and optionally momentum) stored as
//                               bf16, rounded once per call either to nearest even or
//                               stochastically (round up in magnitude with probability equal to
//                               the discarded fraction), the random bits from the counter-based
//                               generator below.
//   * synthetic gradients     - not in the paper: a counter-based generator (Philox4x32-10,
//                               Salmon et al., SC'11) feeding a Box-Muller transform stands in
//                               for forward/backward; each side implements it from the
//                               published definition.
//
// Parity pins (tests/test_oracle_*.py): every function below is pinned against something
// other than itself - closed forms, library routines (numpy quantile / mean, scipy normal pdf,
// torch.optim.SGD, an independent library Philox), brute-force enumeration and the values that
// follow from Eq. 8 for the paper's two heterogeneity vectors.  Nothing here is "parity
// unpinned" except what the paper measures on CIFAR-10 (accuracy / time), which is not
// reproduced here.
//
// Precision: parameters and momentum are fp32 with the fused-multiply-add placement spelled
// out below (compiled with -ffp-contract=off so that only the explicit fmaf calls fuse);
// normals are evaluated in double and rounded once to float; selection is double throughout;
// statistics are summed in double.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <algorithm>
#include <vector>

// The oracle as it stands is single-threaded.  A second build with -fopenmp (oracle/build.py,
// build(openmp=True)) runs the same loops split over column blocks on all host cores, only to time
// an all-cores CPU baseline: every operation is elementwise in the column index, so the results
// are identical bit for bit (tests/test_oracle_openmp.py); the statistics are split over replicas,
// each summed sequentially as before.  Without -fopenmp the macro below is empty.
#ifdef _OPENMP
#include <omp.h>
#define ORACLE_PARALLEL_FOR _Pragma("omp parallel for schedule(static)")
#else
#define ORACLE_PARALLEL_FOR
#endif

namespace {

// ---------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3").
// One round: two 32x32->64 multiplies of counter words 0 and 2 by fixed multipliers; the high
// halves are xored with the other counter words and the round key, the low halves pass through
// (with the word permutation of the definition).  The key is bumped by the Weyl constants
// between rounds.
// ---------------------------------------------------------------------------------------
const uint32_t kMul0 = 0xD2511F53u;
const uint32_t kMul1 = 0xCD9E8D57u;
const uint32_t kWeyl0 = 0x9E3779B9u;  // golden ratio
const uint32_t kWeyl1 = 0xBB67AE85u;  // sqrt(3) - 1

void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    if (round > 0) {
      k0 += kWeyl0;
      k1 += kWeyl1;
    }
    const uint64_t prod0 = (uint64_t)kMul0 * c0;
    const uint64_t prod1 = (uint64_t)kMul1 * c2;
    const uint32_t hi0 = (uint32_t)(prod0 >> 32), lo0 = (uint32_t)prod0;
    const uint32_t hi1 = (uint32_t)(prod1 >> 32), lo1 = (uint32_t)prod1;
    const uint32_t n0 = hi1 ^ c1 ^ k0;
    const uint32_t n1 = lo1;
    const uint32_t n2 = hi0 ^ c3 ^ k1;
    const uint32_t n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Stream tags (word 3 of the counter, top byte).  The low 24 bits of word 3 carry the high
// part of a 56-bit index where one is needed.
const uint32_t kTagInit = 0x49000000u;
const uint32_t kTagGrad = 0x47000000u;
const uint32_t kTagSelect = 0x53000000u;
const uint32_t kTagRound = 0x52000000u;

// Four 32-bit words -> four standard normals (Box-Muller, two pairs).
// u = (x + 0.5) * 2^-32 lies strictly inside (0,1), so the logarithm is finite.
void words_to_normals(const uint32_t x[4], double zd[4]) {
  const double two_pi = 6.283185307179586476925286766559;
  const double scale = 1.0 / 4294967296.0;
  for (int pair = 0; pair < 2; ++pair) {
    const double u0 = ((double)x[2 * pair] + 0.5) * scale;
    const double u1 = ((double)x[2 * pair + 1] + 0.5) * scale;
    const double r = std::sqrt(-2.0 * std::log(u0));
    zd[2 * pair] = r * std::cos(two_pi * u1);
    zd[2 * pair + 1] = r * std::sin(two_pi * u1);
  }
}

void key_of(uint64_t seed, uint32_t key[2]) {
  key[0] = (uint32_t)seed;
  key[1] = (uint32_t)(seed >> 32);
}

// Normals for the four elements 4*group .. 4*group+3 of device `device` at local step `step`.
void grad_normals(uint64_t seed, uint32_t group, uint64_t step, uint32_t device, float z[4]) {
  uint32_t key[2];
  key_of(seed, key);
  const uint32_t ctr[4] = {group, (uint32_t)step, device,
                           kTagGrad | (uint32_t)((step >> 32) & 0xFFFFFFu)};
  uint32_t x[4];
  philox4x32_10(ctr, key, x);
  double zd[4];
  words_to_normals(x, zd);
  for (int i = 0; i < 4; ++i) z[i] = (float)zd[i];
}

// Normals for the initial model (shared by all devices, Algorithm 1 step 1).
void init_normals(uint64_t seed, uint32_t group, float z[4]) {
  uint32_t key[2];
  key_of(seed, key);
  const uint32_t ctr[4] = {group, 0u, 0u, kTagInit};
  uint32_t x[4];
  philox4x32_10(ctr, key, x);
  double zd[4];
  words_to_normals(x, zd);
  for (int i = 0; i < 4; ++i) z[i] = (float)zd[i];
}

// 64 random bits for draw t of selection round `round`.
uint64_t select_bits(uint64_t seed, int64_t round, uint32_t t) {
  uint32_t key[2];
  key_of(seed, key);
  const uint64_t r = (uint64_t)round;
  const uint32_t ctr[4] = {t, 0u, (uint32_t)r, kTagSelect | (uint32_t)((r >> 32) & 0xFFFFFFu)};
  uint32_t x[4];
  philox4x32_10(ctr, key, x);
  return ((uint64_t)x[1] << 32) | (uint64_t)x[0];
}

// bf16 storage: round-to-nearest-even of an fp32 value to the upper 16 bits.
float round_to_bf16(float v) {
  uint32_t bits;
  std::memcpy(&bits, &v, 4);
  if ((bits & 0x7F800000u) == 0x7F800000u) {  // inf / nan: truncate, keep nan a nan
    if (bits & 0x007FFFFFu) bits |= 0x00400000u;
    bits &= 0xFFFF0000u;
  } else {
    const uint32_t lsb = (bits >> 16) & 1u;
    bits += 0x7FFFu + lsb;
    bits &= 0xFFFF0000u;
  }
  float out;
  std::memcpy(&out, &bits, 4);
  return out;
}

// bf16 storage, stochastic rounding: the 16 random bits r are added to the fp32 bit pattern below
// the bf16 mantissa and the sum is truncated, so a finite value moves to its neighbour of larger
// magnitude with probability (discarded 16 bits) / 2^16 and keeps its truncation otherwise; the
// expectation is the value itself.  Infinities and NaNs take the nearest-even path.
float round_to_bf16_stochastic(float v, uint32_t r16) {
  uint32_t bits;
  std::memcpy(&bits, &v, 4);
  if ((bits & 0x7F800000u) == 0x7F800000u) return round_to_bf16(v);
  bits += (r16 & 0xFFFFu);
  bits &= 0xFFFF0000u;
  float out;
  std::memcpy(&out, &bits, 4);
  return out;
}

// Random words for the stochastic rounding at the end of a local-update call: one generator block
// per column group, indexed like the gradient block of the call's last step but with its own tag.
// Element `lane` of the group uses word `lane`: low half for the parameter, high half for the
// momentum.
void rounding_words(uint64_t seed, uint32_t group, uint64_t last_step, uint32_t device,
                    uint32_t x[4]) {
  uint32_t key[2];
  key_of(seed, key);
  const uint32_t ctr[4] = {group, (uint32_t)last_step, device,
                           kTagRound | (uint32_t)((last_step >> 32) & 0xFFFFFFu)};
  philox4x32_10(ctr, key, x);
}

// ---------------------------------------------------------------------------------------
// Selection (Eq. 8).
// ---------------------------------------------------------------------------------------

// Third quartile by linear interpolation between order statistics.
double third_quartile(std::vector<double> xs) {
  std::sort(xs.begin(), xs.end());
  const size_t n = xs.size();
  if (n == 1) return xs[0];
  const double h = 0.75 * (double)(n - 1);
  const size_t lo = (size_t)std::floor(h);
  const double frac = h - (double)lo;
  if (lo + 1 >= n) return xs[n - 1];
  return xs[lo] + frac * (xs[lo + 1] - xs[lo]);
}

// Unnormalised weights f(x_i) / max f, for the available devices; 0 for the others.
// Working with exp(l_i - max l) keeps at least one weight equal to 1 however far the versions
// spread; the common factor cancels in P(i).
void selection_weights(const double* x, const uint8_t* avail, int n, std::vector<double>& wgt) {
  wgt.assign(n, 0.0);
  std::vector<double> xs;
  for (int i = 0; i < n; ++i)
    if (avail[i]) xs.push_back(x[i]);
  if (xs.empty()) return;
  const double mu = third_quartile(xs);
  std::vector<double> l(n, 0.0);
  double lmax = -INFINITY;
  for (int i = 0; i < n; ++i) {
    if (!avail[i]) continue;
    const double d = x[i] - mu;
    l[i] = -(d * d) / 2.0;
    if (l[i] > lmax) lmax = l[i];
  }
  for (int i = 0; i < n; ++i)
    if (avail[i]) wgt[i] = std::exp(l[i] - lmax);
}

void selection_probs(const double* x, const uint8_t* avail, int n, double* P) {
  std::vector<double> wgt;
  selection_weights(x, avail, n, wgt);
  double W = 0.0;
  for (int i = 0; i < n; ++i)
    if (avail[i]) W += wgt[i];
  for (int i = 0; i < n; ++i) P[i] = avail[i] ? wgt[i] / W : 0.0;
}

// Draw k distinct available devices, one after the other, each with probability proportional
// to its weight among those still remaining.  Output in draw order.
int selection_draw(const double* x, const uint8_t* avail, int n, int64_t round, uint64_t seed,
                   int k, int32_t* out) {
  int n_avail = 0;
  for (int i = 0; i < n; ++i) n_avail += avail[i] ? 1 : 0;
  if (k < 1 || k > n_avail) return 1;
  std::vector<double> wgt;
  selection_weights(x, avail, n, wgt);
  std::vector<uint8_t> remaining(avail, avail + n);
  for (int t = 0; t < k; ++t) {
    const uint64_t bits = select_bits(seed, round, (uint32_t)t);
    double W = 0.0;
    int n_rem = 0;
    for (int i = 0; i < n; ++i)
      if (remaining[i]) {
        W += wgt[i];
        ++n_rem;
      }
    int pick = -1;
    if (W > 0.0) {
      const double u = (double)(bits >> 11) * (1.0 / 9007199254740992.0);  // 2^-53
      const double target = u * W;
      double c = 0.0;
      int last_positive = -1;
      for (int i = 0; i < n; ++i) {
        if (!remaining[i]) continue;
        if (wgt[i] > 0.0) last_positive = i;
        c += wgt[i];
        if (c > target) {
          pick = i;
          break;
        }
      }
      if (pick < 0) pick = last_positive;
    } else {
      // every remaining weight underflowed: stragglers are not discarded, pick uniformly.
      int idx = (int)(bits % (uint64_t)n_rem);
      for (int i = 0; i < n; ++i) {
        if (!remaining[i]) continue;
        if (idx == 0) {
          pick = i;
          break;
        }
        --idx;
      }
    }
    remaining[pick] = 0;
    out[t] = pick;
  }
  return 0;
}

// ---------------------------------------------------------------------------------------
// The simulated system: N device replicas over a set of column groups (4 columns each).
// Every operation of the round is elementwise in the column index and selection never looks
// at parameters, so a simulation over any subset of column groups reproduces exactly those
// columns of the full system.
// ---------------------------------------------------------------------------------------
struct Sim {
  int n_devices = 0;
  int64_t n_params = 0;
  int dtype = 0;     // 0: fp32 storage of w, 1: bf16 storage of w
  int m_dtype = 0;   // 0: fp32 storage of the momentum, 1: bf16 (only with bf16 w)
  int rounding = 0;  // bf16 stores of the local update: 0 nearest even, 1 stochastic
  float momentum = 0.f, weight_decay = 0.f, grad_std = 0.f, init_std = 0.f;
  uint64_t seed = 0;
  double version_scale = 1.0;
  int weight_mode = 0;
  std::vector<uint32_t> groups;  // global group index of each held group, ascending
  int64_t n_cols = 0;            // 4 * groups.size()
  std::vector<float> w, m;       // [n_devices][n_cols]; lanes with column >= n_params stay 0
  std::vector<uint32_t> version;
  std::vector<uint64_t> step_count;
  std::vector<uint8_t> avail;

  float* wrow(int i) { return w.data() + (size_t)i * n_cols; }
  float* mrow(int i) { return m.data() + (size_t)i * n_cols; }
  bool live(int64_t g_local, int lane) const {
    return (int64_t)groups[g_local] * 4 + lane < n_params;
  }
};

bool ids_valid(const Sim* s, const int32_t* ids, int n) {
  if (n < 1 || n > s->n_devices) return false;
  std::vector<uint8_t> seen(s->n_devices, 0);
  for (int j = 0; j < n; ++j) {
    if (ids[j] < 0 || ids[j] >= s->n_devices || seen[ids[j]]) return false;
    seen[ids[j]] = 1;
  }
  return true;
}

void scaled_versions(const Sim* s, const double* versions, std::vector<double>& x) {
  x.resize(s->n_devices);
  for (int i = 0; i < s->n_devices; ++i)
    x[i] = (versions ? versions[i] : (double)s->version[i]) * s->version_scale;
}

// Aggregation weights a_j.
// Mode 0 (the paper, Eq. 5 with K = number of selected devices): a_j = 1/k.
// Mode 1 (an extension, not in the paper): a_j proportional to f(x_sel_j), the same f and mu
// as Eq. 8; the last weight is 1 minus the float sum of the others so that they sum to 1.
void aggregation_weights(const Sim* s, const int32_t* sel, int k, const double* versions,
                         float* a) {
  if (s->weight_mode == 0 || k == 1) {
    for (int j = 0; j < k; ++j) a[j] = (float)(1.0 / (double)k);
    return;
  }
  std::vector<double> x;
  scaled_versions(s, versions, x);
  std::vector<double> xs;
  for (int i = 0; i < s->n_devices; ++i)
    if (s->avail[i]) xs.push_back(x[i]);
  const double mu = third_quartile(xs);
  std::vector<double> l(k);
  double lmax = -INFINITY;
  for (int j = 0; j < k; ++j) {
    const double d = x[sel[j]] - mu;
    l[j] = -(d * d) / 2.0;
    lmax = std::max(lmax, l[j]);
  }
  std::vector<double> b(k);
  double B = 0.0;
  for (int j = 0; j < k; ++j) {
    b[j] = std::exp(l[j] - lmax);
    B += b[j];
  }
  float partial = 0.f;
  for (int j = 0; j < k - 1; ++j) {
    a[j] = (float)(b[j] / B);
    partial = partial + a[j];
  }
  a[k - 1] = 1.0f - partial;
}

}  // namespace

extern "C" {

// Threads the loops above run on: 1 in the plain build.
int oracle_threads() {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// ---- generator primitives (exposed for pins and for bit-level comparison) ----------------
void oracle_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
  philox4x32_10(ctr, key, out);
}
void oracle_words_to_normals(const uint32_t* words, double* z) { words_to_normals(words, z); }
void oracle_grad_normals(uint64_t seed, uint32_t group, uint64_t step, uint32_t device, float* z) {
  grad_normals(seed, group, step, device, z);
}
void oracle_init_normals(uint64_t seed, uint32_t group, float* z) { init_normals(seed, group, z); }
uint64_t oracle_select_bits(uint64_t seed, int64_t round, uint32_t t) {
  return select_bits(seed, round, t);
}
float oracle_round_to_bf16(float v) { return round_to_bf16(v); }
float oracle_round_to_bf16_stochastic(float v, uint32_t r16) {
  return round_to_bf16_stochastic(v, r16);
}
void oracle_rounding_words(uint64_t seed, uint32_t group, uint64_t last_step, uint32_t device,
                           uint32_t* x) {
  rounding_words(seed, group, last_step, device, x);
}

// ---- selection without a simulation (Eq. 8) -------------------------------------------------
double oracle_third_quartile(const double* x, int n) {
  return third_quartile(std::vector<double>(x, x + n));
}
void oracle_select_probs(const double* x, const uint8_t* avail, int n, double* P) {
  std::vector<uint8_t> all(n, 1);
  selection_probs(x, avail ? avail : all.data(), n, P);
}
int oracle_select(const double* x, const uint8_t* avail, int n, int64_t round, uint64_t seed,
                  int k, int32_t* out) {
  std::vector<uint8_t> all(n, 1);
  return selection_draw(x, avail ? avail : all.data(), n, round, seed, k, out);
}

// ---- version prediction (Eq. 7) ---------------------------------------------------------------
// Brown's double exponential smoothing over the observed series v[0..n_obs-1]; both smoothed
// series start at the first observation.  Returns the prediction m rounds after the last one.
double oracle_predict_version(const double* v, int n_obs, double alpha, double m) {
  double s1 = v[0], s2 = v[0];
  for (int j = 1; j < n_obs; ++j) {
    s1 = alpha * v[j] + (1.0 - alpha) * s1;
    s2 = alpha * s1 + (1.0 - alpha) * s2;
  }
  const double a = 2.0 * s1 - s2;
  const double b = alpha / (1.0 - alpha) * (s1 - s2);
  return a + b * m;
}

// ---- the simulated system -------------------------------------------------------------------
// groups == NULL: hold every column group of the model.
void* oracle_sim_create(int n_devices, int64_t n_params, int dtype, float momentum,
                        float weight_decay, float grad_std, float init_std, uint64_t seed,
                        double version_scale, int weight_mode, const uint32_t* groups,
                        int64_t n_groups, int m_dtype, int rounding) {
  if (n_devices < 1 || n_params < 1 || (dtype != 0 && dtype != 1)) return nullptr;
  if ((m_dtype != 0 && m_dtype != 1) || (rounding != 0 && rounding != 1)) return nullptr;
  if (dtype == 0 && (m_dtype != 0 || rounding != 0)) return nullptr;  // bf16 options need bf16 w
  Sim* s = new Sim;
  s->m_dtype = m_dtype;
  s->rounding = rounding;
  s->n_devices = n_devices;
  s->n_params = n_params;
  s->dtype = dtype;
  s->momentum = momentum;
  s->weight_decay = weight_decay;
  s->grad_std = grad_std;
  s->init_std = init_std;
  s->seed = seed;
  s->version_scale = version_scale;
  s->weight_mode = weight_mode;
  const int64_t all_groups = (n_params + 3) / 4;
  if (groups) {
    s->groups.assign(groups, groups + n_groups);
    for (uint32_t g : s->groups)
      if ((int64_t)g >= all_groups) {
        delete s;
        return nullptr;
      }
  } else {
    s->groups.resize(all_groups);
    for (int64_t g = 0; g < all_groups; ++g) s->groups[g] = (uint32_t)g;
  }
  s->n_cols = 4 * (int64_t)s->groups.size();
  s->w.assign((size_t)n_devices * s->n_cols, 0.f);
  s->m.assign((size_t)n_devices * s->n_cols, 0.f);
  s->version.assign(n_devices, 0u);
  s->step_count.assign(n_devices, 0ull);
  s->avail.assign(n_devices, 1);
  // Algorithm 1, step 1: every device starts from the same w_(0) = init_std * z.
  for (int64_t gl = 0; gl < (int64_t)s->groups.size(); ++gl) {
    float z[4];
    init_normals(seed, s->groups[gl], z);
    for (int lane = 0; lane < 4; ++lane) {
      if (!s->live(gl, lane)) continue;
      float v = init_std * z[lane];
      if (dtype == 1) v = round_to_bf16(v);
      for (int i = 0; i < n_devices; ++i) s->wrow(i)[4 * gl + lane] = v;
    }
  }
  return s;
}

void oracle_sim_destroy(void* p) { delete (Sim*)p; }

int64_t oracle_sim_n_cols(void* p) { return ((Sim*)p)->n_cols; }

// Local update (Eq. 3 / Algorithm 1): device ids[j] runs steps[j] SGD steps on its own replica.
//   g  = grad_std * z + wd * w      (one rounding for the product grad_std*z, then one fma)
//   m  = mu * m + g                 (one fma)
//   w  = w - lr * m                 (one fma)
// With bf16 storage a value is widened on entry, kept in fp32 through the steps of this call and
// rounded once at its end (to nearest even, or stochastically with the words of rounding_words).
// A device that runs no step in the call is not touched at all.
int oracle_sim_local_step(void* p, const int32_t* ids, const int32_t* steps, int n, float lr) {
  Sim* s = (Sim*)p;
  if (!ids || !steps || !ids_valid(s, ids, n)) return 1;
  for (int j = 0; j < n; ++j)
    if (steps[j] < 0) return 1;
  for (int j = 0; j < n; ++j) {
    const int dev = ids[j];
    float* w = s->wrow(dev);
    float* m = s->mrow(dev);
    ORACLE_PARALLEL_FOR
    for (int64_t gl = 0; gl < (int64_t)s->groups.size(); ++gl) {
      for (int e = 0; e < steps[j]; ++e) {
        float z[4];
        grad_normals(s->seed, s->groups[gl], s->step_count[dev] + (uint64_t)e, (uint32_t)dev, z);
        for (int lane = 0; lane < 4; ++lane) {
          if (!s->live(gl, lane)) continue;
          const int64_t c = 4 * gl + lane;
          const float noise = s->grad_std * z[lane];
          const float g = std::fmaf(s->weight_decay, w[c], noise);
          m[c] = std::fmaf(s->momentum, m[c], g);
          w[c] = std::fmaf(-lr, m[c], w[c]);
        }
      }
      if (s->dtype == 1 && steps[j] > 0) {
        uint32_t x[4] = {0u, 0u, 0u, 0u};
        if (s->rounding == 1)
          rounding_words(s->seed, s->groups[gl], s->step_count[dev] + (uint64_t)steps[j] - 1,
                         (uint32_t)dev, x);
        for (int lane = 0; lane < 4; ++lane) {
          const int64_t c = 4 * gl + lane;
          if (s->rounding == 1) {
            w[c] = round_to_bf16_stochastic(w[c], x[lane] & 0xFFFFu);
            if (s->m_dtype == 1) m[c] = round_to_bf16_stochastic(m[c], x[lane] >> 16);
          } else {
            w[c] = round_to_bf16(w[c]);
            if (s->m_dtype == 1) m[c] = round_to_bf16(m[c]);
          }
        }
      }
    }
    s->step_count[dev] += (uint64_t)steps[j];
    s->version[dev] += (uint32_t)steps[j];
  }
  return 0;
}

int oracle_sim_select_probs(void* p, const double* versions, double* P) {
  Sim* s = (Sim*)p;
  std::vector<double> x;
  scaled_versions(s, versions, x);
  int n_avail = 0;
  for (uint8_t a : s->avail) n_avail += a;
  if (n_avail == 0) return 1;
  selection_probs(x.data(), s->avail.data(), s->n_devices, P);
  return 0;
}

int oracle_sim_select(void* p, int64_t round, const double* versions, uint64_t seed, int k,
                      int32_t* out) {
  Sim* s = (Sim*)p;
  std::vector<double> x;
  scaled_versions(s, versions, x);
  return selection_draw(x.data(), s->avail.data(), s->n_devices, round, seed, k, out);
}

int oracle_sim_aggregation_weights(void* p, const int32_t* sel, int k, const double* versions,
                                   float* a) {
  Sim* s = (Sim*)p;
  if (!sel || !ids_valid(s, sel, k)) return 1;
  aggregation_weights(s, sel, k, versions, a);
  return 0;
}

// Partial aggregation (Eq. 5) with write-back to the selected replicas:
//   acc = a_0 * w[sel_0];  acc = fma(a_j, w[sel_j], acc) for j = 1..k-1 in the order of `sel`.
// Momentum is local to a device and is not touched.  The aggregated model carries the newest
// version among its inputs.
int oracle_sim_aggregate(void* p, const int32_t* sel, int k, const double* versions) {
  Sim* s = (Sim*)p;
  if (!sel || !ids_valid(s, sel, k)) return 1;
  std::vector<float> a(k);
  aggregation_weights(s, sel, k, versions, a.data());
  ORACLE_PARALLEL_FOR
  for (int64_t c = 0; c < s->n_cols; ++c) {
    float acc = a[0] * s->wrow(sel[0])[c];
    for (int j = 1; j < k; ++j) acc = std::fmaf(a[j], s->wrow(sel[j])[c], acc);
    if (s->dtype == 1) acc = round_to_bf16(acc);
    for (int j = 0; j < k; ++j) s->wrow(sel[j])[c] = acc;
  }
  uint32_t vmax = 0;
  for (int j = 0; j < k; ++j) vmax = std::max(vmax, s->version[sel[j]]);
  for (int j = 0; j < k; ++j) s->version[sel[j]] = vmax;
  return 0;
}

// Global synchronisation (Algorithm 1: send the aggregate to devices whose Flag is 0): the
// receivers' parameters are overwritten by the sender's and take its version.
int oracle_sim_broadcast(void* p, int src, const int32_t* dst, int n) {
  Sim* s = (Sim*)p;
  if (src < 0 || src >= s->n_devices) return 1;
  if (n == 0) return 0;
  if (!dst || !ids_valid(s, dst, n)) return 1;
  for (int j = 0; j < n; ++j)
    if (dst[j] == src) return 1;
  for (int j = 0; j < n; ++j) {
    std::memcpy(s->wrow(dst[j]), s->wrow(src), sizeof(float) * (size_t)s->n_cols);
    s->version[dst[j]] = s->version[src];
  }
  return 0;
}

// Global synchronisation read as a mix (Section "Model aggregation and fault-tolerant": the
// unselected devices fold the received model into their own before the next local steps; the
// paper gives no formula).  Reading offered beside the overwrite of Algorithm 1: a convex
// combination with weight beta on the received model,
//     w_dst = beta * w_src + (1 - beta) * w_dst,
// evaluated as  t = (1 - beta) * w_dst  (1 - beta and the product rounded to float), then one fused
// multiply-add  fma(beta, w_src, t).  beta = 1 reproduces the overwrite, beta = 0 leaves the
// receiver as it is.  With bf16 storage the result is rounded to nearest even.  The receiver's
// version becomes the larger of the two (it now carries both lineages), or the sender's when
// beta = 1 (nothing of its own remains).
int oracle_sim_integrate(void* p, int src, const int32_t* dst, int n, float beta) {
  Sim* s = (Sim*)p;
  if (src < 0 || src >= s->n_devices) return 1;
  if (!(beta >= 0.0f && beta <= 1.0f)) return 1;
  if (n == 0) return 0;
  if (!dst || !ids_valid(s, dst, n)) return 1;
  for (int j = 0; j < n; ++j)
    if (dst[j] == src) return 1;
  const float one_minus_beta = 1.0f - beta;
  const float* from = s->wrow(src);
  for (int j = 0; j < n; ++j) {
    float* to = s->wrow(dst[j]);
    ORACLE_PARALLEL_FOR
    for (int64_t c = 0; c < s->n_cols; ++c) {
      const float t = one_minus_beta * to[c];
      const float v = std::fmaf(beta, from[c], t);
      to[c] = s->dtype == 1 ? round_to_bf16(v) : v;
    }
    if (beta == 1.0f)
      s->version[dst[j]] = s->version[src];
    else if (s->version[src] > s->version[dst[j]])
      s->version[dst[j]] = s->version[src];
  }
  return 0;
}

// Per-replica squared norm and squared distance to a reference replica, over the held columns.
int oracle_sim_stats(void* p, int ref, double* norm2, double* div2) {
  Sim* s = (Sim*)p;
  if (ref < 0 || ref >= s->n_devices) return 1;
  ORACLE_PARALLEL_FOR
  for (int i = 0; i < s->n_devices; ++i) {
    double n2 = 0.0, d2 = 0.0;
    for (int64_t c = 0; c < s->n_cols; ++c) {
      const double wi = (double)s->wrow(i)[c];
      const double d = wi - (double)s->wrow(ref)[c];
      n2 += wi * wi;
      d2 += d * d;
    }
    norm2[i] = n2;
    div2[i] = d2;
  }
  return 0;
}

// which: 0 = parameters, 1 = momentum.  Copies the held columns (4 per group, group order).
int oracle_sim_read(void* p, int id, int which, float* dst) {
  Sim* s = (Sim*)p;
  if (id < 0 || id >= s->n_devices) return 1;
  std::memcpy(dst, which ? s->mrow(id) : s->wrow(id), sizeof(float) * (size_t)s->n_cols);
  return 0;
}

int oracle_sim_write(void* p, int id, int which, const float* src) {
  Sim* s = (Sim*)p;
  if (id < 0 || id >= s->n_devices) return 1;
  float* row = which ? s->mrow(id) : s->wrow(id);
  for (int64_t gl = 0; gl < (int64_t)s->groups.size(); ++gl)
    for (int lane = 0; lane < 4; ++lane) {
      const int64_t c = 4 * gl + lane;
      if (!s->live(gl, lane)) continue;
      const bool narrow = which == 0 ? s->dtype == 1 : s->m_dtype == 1;
      row[c] = narrow ? round_to_bf16(src[c]) : src[c];
    }
  return 0;
}

void oracle_sim_get_versions(void* p, uint32_t* versions, uint64_t* step_counts) {
  Sim* s = (Sim*)p;
  for (int i = 0; i < s->n_devices; ++i) {
    if (versions) versions[i] = s->version[i];
    if (step_counts) step_counts[i] = s->step_count[i];
  }
}

void oracle_sim_set_versions(void* p, const uint32_t* versions, const uint64_t* step_counts) {
  Sim* s = (Sim*)p;
  for (int i = 0; i < s->n_devices; ++i) {
    if (versions) s->version[i] = versions[i];
    if (step_counts) s->step_count[i] = step_counts[i];
  }
}

void oracle_sim_set_available(void* p, const uint8_t* mask) {
  Sim* s = (Sim*)p;
  for (int i = 0; i < s->n_devices; ++i) s->avail[i] = mask ? (mask[i] ? 1 : 0) : 1;
}

}  // extern "C"
