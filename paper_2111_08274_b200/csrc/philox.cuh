// Counter-based random numbers for the synthetic gradients, the initial model and the selection
// draws: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3",
// SC'11), written from that paper's definition.  The ten round keys depend only on the run's
// seed, so the host expands them once and the kernels receive them as launch parameters
// (constant bank): the device code spends no instruction on the key schedule.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define HADFL_HD __host__ __device__ __forceinline__
#else
#define HADFL_HD inline
#endif

namespace hadfl {

constexpr uint32_t kPhiloxM0 = 0xD2511F53u;
constexpr uint32_t kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u;
constexpr uint32_t kPhiloxW1 = 0xBB67AE85u;

// Stream tags: top byte of counter word 3; its low 24 bits extend word 1 / word 2 to 56 bits.
constexpr uint32_t kTagInit = 0x49000000u;    // 'I': initial model, counter (group, 0, 0, tag)
constexpr uint32_t kTagGrad = 0x47000000u;    // 'G': gradients, counter (group, step, device, tag|step>>32)
constexpr uint32_t kTagSelect = 0x53000000u;  // 'S': selection, counter (draw, 0, round, tag|round>>32)
constexpr uint32_t kTagRound = 0x52000000u;   // 'R': stochastic rounding, counter (group, last step, device, tag|step>>32)

struct PhiloxKeys {
  uint32_t a[10];  // round keys for the word-0 product
  uint32_t b[10];  // round keys for the word-2 product
};

inline PhiloxKeys expand_keys(uint64_t seed) {
  PhiloxKeys k;
  uint32_t a = (uint32_t)seed, b = (uint32_t)(seed >> 32);
  for (int r = 0; r < 10; ++r) {
    k.a[r] = a;
    k.b[r] = b;
    a += kPhiloxW0;
    b += kPhiloxW1;
  }
  return k;
}

HADFL_HD void philox_round(uint32_t &c0, uint32_t &c1, uint32_t &c2, uint32_t &c3, uint32_t ka,
                           uint32_t kb) {
  const unsigned long long p0 = (unsigned long long)kPhiloxM0 * c0;
  const unsigned long long p1 = (unsigned long long)kPhiloxM1 * c2;
  const uint32_t t0 = (uint32_t)(p1 >> 32) ^ c1 ^ ka;
  const uint32_t t2 = (uint32_t)(p0 >> 32) ^ c3 ^ kb;
  c1 = (uint32_t)p1;
  c3 = (uint32_t)p0;
  c0 = t0;
  c2 = t2;
}

HADFL_HD void philox4x32_10(uint32_t &c0, uint32_t &c1, uint32_t &c2, uint32_t &c3,
                            const PhiloxKeys &k) {
#pragma unroll
  for (int r = 0; r < 10; ++r) philox_round(c0, c1, c2, c3, k.a[r], k.b[r]);
}

}  // namespace hadfl
