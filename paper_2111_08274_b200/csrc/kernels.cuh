// sm_100a kernels of the HADFL round: initial model (K0), batched heterogeneity-aware local
// update (K1; Eq. 3 / Algorithm 1), fused weighted aggregation with write-back (K2; Eq. 5),
// the mix of a received model into the receivers' own (Section "Model aggregation and
// fault-tolerant"), per-replica statistics (K3), and the fused round (K1 + K2 + global
// synchronisation + K3 in one pass over the arena).
//
// All of them stream rows of one [N][stride] arena.  A "column group" is four consecutive
// parameters (one Philox block); a thread holds a "pack" of a row - 16 bytes of w in K2 / K3,
// eight parameters in K1 and the fused round - and walks over the rows, so that
//   - accesses of a warp are contiguous (512 bytes per 128-bit load instruction),
//   - several independent row loads are in flight per thread before the first dependent use
//     (loads fill raw packs; widening bf16 to fp32 happens where the values are used),
//   - every thread does the same amount of arithmetic whatever the per-device step counts are
//     (the kernel-level answer to the straggler problem the paper is about), and
//   - the arithmetic order per element is fixed, hence results are reproducible bit for bit.
// None of this is a dense contraction, so there is no tensor-core path: the bound is HBM
// bandwidth, except for the local update with several steps per device, where instruction issue
// (the integer multiplies of Philox, Box-Muller on the special-function unit) binds.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

#include "debug_check.cuh"
#include "philox.cuh"

namespace hadfl {

constexpr int kMaxDevices = 32;
constexpr int kThreads = 256;

// ------------------------------------------------------------------------------------------
// Storage access by element and by column group (used by the initial-model kernel and by the
// ragged last pack of a row).
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void st_group(float *row, int64_t g, float4 v) {
  if (!access_ok(row + 4 * g, 16)) return;
  *reinterpret_cast<float4 *>(row + 4 * g) = v;
}
__device__ __forceinline__ void st_group(__nv_bfloat16 *row, int64_t g, float4 v) {
  if (!access_ok(row + 4 * g, 8)) return;
  const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
  const __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 raw;
  raw.x = *reinterpret_cast<const uint32_t *>(&lo);
  raw.y = *reinterpret_cast<const uint32_t *>(&hi);
  *reinterpret_cast<uint2 *>(row + 4 * g) = raw;
}
__device__ __forceinline__ void st_elem(float *row, int64_t p, float v) {
  if (access_ok(row + p, 4)) row[p] = v;
}
__device__ __forceinline__ void st_elem(__nv_bfloat16 *row, int64_t p, float v) {
  if (access_ok(row + p, 2)) row[p] = __float2bfloat16_rn(v);
}

// ------------------------------------------------------------------------------------------
// Packs: E consecutive parameters held by one thread (E = 4 or 8).  fp32: E/4 128-bit accesses;
// bf16: one 64-bit (E = 4) or 128-bit (E = 8) access.  A pack of 8 is two column groups, i.e.
// two Philox blocks.  `live` < E only in the ragged last pack of a row.
// ------------------------------------------------------------------------------------------
template <typename WT>
struct Pack16 {  // the pack that is 16 bytes of storage
  static constexpr int E = sizeof(WT) == 2 ? 8 : 4;
};

template <int E>
__device__ __forceinline__ void st_pack(float *row, int64_t p, const float (&v)[E]) {
  if (!access_ok(row + E * p, 4 * E)) return;
#pragma unroll
  for (int i = 0; i < E / 4; ++i)
    *reinterpret_cast<float4 *>(row + E * p + 4 * i) =
        make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
}
__device__ __forceinline__ void bf16x2_to_floats(uint32_t raw, float &lo, float &hi) {
  lo = __uint_as_float(raw << 16);
  hi = __uint_as_float(raw & 0xFFFF0000u);
}
__device__ __forceinline__ uint32_t floats_to_bf16x2(float lo, float hi) {
  const __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t *>(&t);
}
template <int E>
__device__ __forceinline__ void st_pack(__nv_bfloat16 *row, int64_t p, const float (&v)[E]) {
  if (!access_ok(row + E * p, 2 * E)) return;
  if (E == 8) {
    uint4 raw;
    raw.x = floats_to_bf16x2(v[0], v[1]);
    raw.y = floats_to_bf16x2(v[2], v[3]);
    raw.z = floats_to_bf16x2(v[E - 4], v[E - 3]);
    raw.w = floats_to_bf16x2(v[E - 2], v[E - 1]);
    *reinterpret_cast<uint4 *>(row + 8 * p) = raw;
  } else {
    uint2 raw;
    raw.x = floats_to_bf16x2(v[0], v[1]);
    raw.y = floats_to_bf16x2(v[2], v[3]);
    *reinterpret_cast<uint2 *>(row + 4 * p) = raw;
  }
}
// A loaded pack as it came from memory.  Loads fill a RawPack and nothing else, so that a thread
// can issue all the loads of a batch (or both loads of a row) without an instruction that
// depends on the data in between; `unpack` widens to fp32 registers at the point of use.
template <typename WT, int E>
struct RawPack;
template <int E>
struct RawPack<float, E> {
  float v[E];
};
template <>
struct RawPack<__nv_bfloat16, 8> {
  uint4 q;
};
template <>
struct RawPack<__nv_bfloat16, 4> {
  uint2 q;
};

template <int E>
__device__ __forceinline__ void unpack(const RawPack<float, E> &r, float (&v)[E]) {
#pragma unroll
  for (int i = 0; i < E; ++i) v[i] = r.v[i];
}
__device__ __forceinline__ void unpack(const RawPack<__nv_bfloat16, 8> &r, float (&v)[8]) {
  bf16x2_to_floats(r.q.x, v[0], v[1]);
  bf16x2_to_floats(r.q.y, v[2], v[3]);
  bf16x2_to_floats(r.q.z, v[4], v[5]);
  bf16x2_to_floats(r.q.w, v[6], v[7]);
}
__device__ __forceinline__ void unpack(const RawPack<__nv_bfloat16, 4> &r, float (&v)[4]) {
  bf16x2_to_floats(r.q.x, v[0], v[1]);
  bf16x2_to_floats(r.q.y, v[2], v[3]);
}

// `at` points to the first element of the pack.  live == E: vector load; otherwise (the ragged
// last pack of a row) element by element, dead lanes read as 0.
template <int E>
__device__ __forceinline__ void ld_raw(const float *at, int live, RawPack<float, E> &r) {
  if (!access_ok(at, 4 * (size_t)live)) {  // debug build only: a skipped load reads as zeros
#pragma unroll
    for (int i = 0; i < E; ++i) r.v[i] = 0.f;
    return;
  }
  if (live == E) {
#pragma unroll
    for (int i = 0; i < E / 4; ++i) {
      const float4 t = *reinterpret_cast<const float4 *>(at + 4 * i);
      r.v[4 * i] = t.x; r.v[4 * i + 1] = t.y; r.v[4 * i + 2] = t.z; r.v[4 * i + 3] = t.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < E; ++i) r.v[i] = i < live ? at[i] : 0.f;
  }
}
__device__ __forceinline__ uint32_t ld_bf16_bits(const __nv_bfloat16 *at, int i, int live) {
  return i < live ? (uint32_t)*reinterpret_cast<const unsigned short *>(at + i) : 0u;
}
__device__ __forceinline__ void ld_raw(const __nv_bfloat16 *at, int live, RawPack<__nv_bfloat16, 8> &r) {
  if (!access_ok(at, 2 * (size_t)live)) {
    r.q = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  if (live == 8) {
    r.q = *reinterpret_cast<const uint4 *>(at);
  } else {
    r.q.x = ld_bf16_bits(at, 0, live) | (ld_bf16_bits(at, 1, live) << 16);
    r.q.y = ld_bf16_bits(at, 2, live) | (ld_bf16_bits(at, 3, live) << 16);
    r.q.z = ld_bf16_bits(at, 4, live) | (ld_bf16_bits(at, 5, live) << 16);
    r.q.w = ld_bf16_bits(at, 6, live) | (ld_bf16_bits(at, 7, live) << 16);
  }
}
__device__ __forceinline__ void ld_raw(const __nv_bfloat16 *at, int live, RawPack<__nv_bfloat16, 4> &r) {
  if (!access_ok(at, 2 * (size_t)live)) {
    r.q = make_uint2(0u, 0u);
    return;
  }
  if (live == 4) {
    r.q = *reinterpret_cast<const uint2 *>(at);
  } else {
    r.q.x = ld_bf16_bits(at, 0, live) | (ld_bf16_bits(at, 1, live) << 16);
    r.q.y = ld_bf16_bits(at, 2, live) | (ld_bf16_bits(at, 3, live) << 16);
  }
}
template <typename WT, int E>
__device__ __forceinline__ void zero_raw(RawPack<WT, E> &r) {
  memset(&r, 0, sizeof(r));
}
template <typename T, int E>
__device__ __forceinline__ void st_pack_any(T *row, int64_t p, int live, const float (&v)[E]) {
  if (live == E) {
    st_pack<E>(row, p, v);
  } else {
#pragma unroll
    for (int i = 0; i < E; ++i)
      if (i < live) st_elem(row, E * p + i, v[i]);
  }
}
// The value a parameter has once stored: itself for fp32, rounded to nearest even for bf16.
__device__ __forceinline__ float as_stored(float v, const float *) { return v; }
__device__ __forceinline__ float as_stored(float v, const __nv_bfloat16 *) {
  return __bfloat162float(__float2bfloat16_rn(v));
}
__device__ __forceinline__ int live_of(int64_t n_params, int64_t p, int E) {
  const int64_t left = n_params - (int64_t)E * p;
  return left >= E ? E : (left > 0 ? (int)left : 0);
}

// ------------------------------------------------------------------------------------------
// Uniform words -> standard normals (Box-Muller).  (x0, x1) -> (z0, z1):
//   u0 = (x0 + 0.5) 2^-32,  u1 = (x1 + 0.5) 2^-32,  r = sqrt(-2 ln u0),
//   z0 = r cos(2 pi u1),    z1 = r sin(2 pi u1).
// The angle is taken as a = u1 - [x1 >= 2^31] in (-1/2, 1/2), the same angle modulo a turn,
// by reading x1 as a signed integer: small angles keep their relative precision.
// ------------------------------------------------------------------------------------------

// Special-function-unit instructions in their flush-to-zero forms (no subnormal fix-up code; the
// arguments here are never subnormal).
__device__ __forceinline__ float sfu_sqrt(float x) {
  float y;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float sfu_lg2(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float sfu_sin(float x) {
  float y;
  asm("sin.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float sfu_cos(float x) {
  float y;
  asm("cos.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// -2 ln(1 - t) by its series, for t = 1 - u0 = (~x0 + 0.5) 2^-32 < 2^-10, times `scale2`:
// 2t + t^2 + (2/3) t^3 (the next term, t^4/2, is below 2^-31 relative).  Only reached from a rarely
// taken branch (one combined test per step), so the common path pays a compare and an untaken
// branch for it; inlined there, because a real call inside the step loop makes the compiler shuffle
// the live registers around every call site (about one instruction per step on average).
__device__ __forceinline__ float r2_next_to_one(uint32_t x0, float scale2) {
  const float t = fmaf(__uint2float_rn(~x0), 0x1p-32f, 0x1p-33f);
  return scale2 * (t * fmaf(t, fmaf(t, 0.66666667f, 1.0f), 2.0f));
}

struct NormalsFast {
  // The four normals of standard deviation s of one Philox block (words x0 .. x3; pairs (x0, x1)
  // and (x2, x3)); the caller passes lg_scale = -2 ln2 s^2 and scale2 = s^2 so that the scaling
  // costs no instruction:
  //   r^2 = lg_scale * lg2(u0)            (u0 = (x0 + 0.5) 2^-32)
  //   theta = 2 pi a,  a = ((int)x1 + 0.5) 2^-32          (one fused multiply-add)
  // The fp32 arithmetic is written on packed pairs (sm_100's two-wide fp32 instructions: one issue
  // slot, two IEEE results): the block's two radii, its two angles, the two normals of a pair.
  // Next to u0 = 1 (x0 >= 2^32 - 2^22) lg2.approx only has an absolute error bound, so the exact
  // complement and a series take over.  Measured against a double-precision evaluation (s = 1):
  // max |dz| about 2e-6, mean 1.6e-7.
  static constexpr uint32_t kNearOne = 0xFFC00000u;
  // r^2 of both pairs, away from u0 = 1 (wrong by up to a few 1e-7 absolute next to it: see needs_series)
  static __device__ __forceinline__ float2 radius2_pair(uint32_t x0, uint32_t x2, float lg_scale) {
    const float2 u = __ffma2_rn(make_float2(__uint2float_rn(x0), __uint2float_rn(x2)),
                                make_float2(0x1p-32f, 0x1p-32f), make_float2(0x1p-33f, 0x1p-33f));
    return __fmul2_rn(make_float2(lg_scale, lg_scale), make_float2(sfu_lg2(u.x), sfu_lg2(u.y)));
  }
  static __device__ __forceinline__ bool needs_series(uint32_t x0) { return x0 >= kNearOne; }
  // theta of both pairs (words 1 and 3)
  static __device__ __forceinline__ float2 angle_pair(uint32_t x1, uint32_t x3) {
    return __ffma2_rn(make_float2(__int2float_rn((int)x1), __int2float_rn((int)x3)),
                      make_float2(1.4629180792671596e-9f, 1.4629180792671596e-9f),
                      make_float2(7.314590396335798e-10f, 7.314590396335798e-10f));
  }
  // (r cos theta, r sin theta)
  static __device__ __forceinline__ float2 finish_pair(float r2, float theta) {
    const float r = sfu_sqrt(r2);
    return __fmul2_rn(make_float2(r, r), make_float2(sfu_cos(theta), sfu_sin(theta)));
  }
  static __device__ __forceinline__ float4 block(uint32_t x0, uint32_t x1, uint32_t x2, uint32_t x3,
                                                 float lg_scale, float scale2) {
    float2 r2 = radius2_pair(x0, x2, lg_scale);
    if (needs_series(x0)) r2.x = r2_next_to_one(x0, scale2);
    if (needs_series(x2)) r2.y = r2_next_to_one(x2, scale2);
    const float2 theta = angle_pair(x1, x3);
    const float2 z01 = finish_pair(r2.x, theta.x), z23 = finish_pair(r2.y, theta.y);
    return make_float4(z01.x, z01.y, z23.x, z23.y);
  }
};

struct NormalsAccurate {
  // Full-precision fp32 library functions; the logarithm of u0 >= 1/2 is taken through the exact
  // complement 1 - u0 = (~x0 + 0.5) 2^-32 so that it keeps its relative accuracy next to 1.
  static __device__ __forceinline__ void pair(uint32_t x0, uint32_t x1, float lg_scale,
                                              float scale2, float &z0, float &z1) {
    (void)lg_scale;
    float neg_ln;
    if (x0 & 0x80000000u) {
      const float t = fmaf(__uint2float_rn(~x0), 0x1p-32f, 0x1p-33f);
      neg_ln = -log1pf(-t);
    } else {
      const float u0 = fmaf(__uint2float_rn(x0), 0x1p-32f, 0x1p-33f);
      neg_ln = -logf(u0);
    }
    const float a = fmaf(__int2float_rn((int)x1), 0x1p-32f, 0x1p-33f);
    const float r = sqrtf(2.0f * scale2 * neg_ln);
    float s, c;
    sincospif(2.0f * a, &s, &c);
    z0 = r * c;
    z1 = r * s;
  }
  static __device__ __forceinline__ float4 block(uint32_t x0, uint32_t x1, uint32_t x2, uint32_t x3,
                                                 float lg_scale, float scale2) {
    float4 z;
    pair(x0, x1, lg_scale, scale2, z.x, z.y);
    pair(x2, x3, lg_scale, scale2, z.z, z.w);
    return z;
  }
};

constexpr float kMinusTwoLn2 = -1.3862943611198906f;

// Unit normals of one Philox block.
template <typename Gen>
__device__ __forceinline__ float4 normals_of_block(uint32_t c0, uint32_t c1, uint32_t c2,
                                                   uint32_t c3, const PhiloxKeys &keys) {
  philox4x32_10(c0, c1, c2, c3, keys);
  return Gen::block(c0, c1, c2, c3, kMinusTwoLn2, 1.0f);
}

// ------------------------------------------------------------------------------------------
// K0: initial model.  Every row gets w_(0)[p] = init_std * z(seed; p), momentum 0; lanes beyond P
// (ragged group and row padding) are zeroed in both arenas.  One thread per column group of the
// padded row.
// ------------------------------------------------------------------------------------------
template <typename WT, typename MT>
__global__ void __launch_bounds__(kThreads)
k_init(WT *__restrict__ w, MT *__restrict__ m, int64_t stride, int64_t n_params, int n_devices,
       PhiloxKeys keys, float init_std) {
  const int64_t g = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (4 * g >= stride) return;
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (4 * g < n_params) {
    const float4 z = normals_of_block<NormalsAccurate>((uint32_t)g, 0u, 0u, kTagInit, keys);
    v.x = init_std * z.x;
    if (4 * g + 1 < n_params) v.y = init_std * z.y;
    if (4 * g + 2 < n_params) v.z = init_std * z.z;
    if (4 * g + 3 < n_params) v.w = init_std * z.w;
  }
  const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int i = 0; i < n_devices; ++i) {
    st_group(w + (int64_t)i * stride, g, v);
    st_group(m + (int64_t)i * stride, g, zero);
  }
}

// ------------------------------------------------------------------------------------------
// K1: batched local update (Eq. 3 / Algorithm 1) for a list of devices with per-device step
// counts, one launch.  A thread owns a pack of E columns (E/4 Philox blocks) and visits the listed
// rows one after the other: load w and m once, run that device's steps in registers (gradient
// from the counter-based generator), store once; other resident warps cover the load latency.
// The gradient noise grad_std * z is produced directly (the scale is
// folded into the constants of the radius), which differs from rounding z first by about one
// part in 10^7.
//
// The first Philox round of a gradient block multiplies the column-group index (fixed per thread)
// and the device id (fixed per row), so it is hoisted: the host folds the device product, the tag
// word and the first round keys into three words per row, the thread keeps the group product, and
// per step the round is two xors.  The host also guarantees that a row's step counter does not
// cross a multiple of 2^32 inside one launch (it splits the call), so the step index is one add.
// ------------------------------------------------------------------------------------------
struct RowStep {
  int64_t w_off;     // byte offset of the device's row in the parameter arena
  int64_t m_off;     // byte offset of the device's row in the momentum arena
  int32_t row;
  int32_t steps;
  uint32_t base_lo;  // low word of the device's step counter before this call
  uint32_t r1_c0;    // hi(M1 * device) ^ key_a[0]      (xor step index -> word 0)
  uint32_t r1_c1;    // lo(M1 * device)                                 (word 1)
  uint32_t r1_c2;    // (tag | step_hi) ^ key_b[0]   (xor hi(M0 * group) -> word 2)
};

struct LocalStepArgs {  // the host lists only devices that run at least one step
  int32_t n;
  RowStep r[kMaxDevices];
};

// Constants of the update, computed once on the host and read from the launch parameters:
// -lr, momentum, weight decay, -2 ln2 grad_std^2 and grad_std^2.
struct StepConsts {
  float neg_lr, mu, wd, lg_scale, scale2;
};

// The thread's share of the first Philox round: hi/lo of M0 * group for each of its NB groups.
template <int NB>
struct GroupProducts {
  uint32_t hi[NB], lo[NB];
  __device__ __forceinline__ explicit GroupProducts(int64_t pack) {
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      const unsigned long long gp = (unsigned long long)kPhiloxM0 * (uint32_t)(pack * NB + b);
      hi[b] = (uint32_t)(gp >> 32);
      lo[b] = (uint32_t)gp;
    }
  }
};

// One SGD step of two parameters on packed pairs:
//   g = fma(wd, w, noise);  m = fma(mu, m, g);  w = fma(-lr, m, w)        (per lane, as in Eq. 3)
__device__ __forceinline__ void sgd_update_pair(float &w0, float &w1, float &m0, float &m1, float2 noise,
                                                float2 wd2, float2 mu2, float2 neg_lr2) {
  const float2 w2 = make_float2(w0, w1);
  const float2 g2 = __ffma2_rn(wd2, w2, noise);
  const float2 m2 = __ffma2_rn(mu2, make_float2(m0, m1), g2);
  const float2 w2n = __ffma2_rn(neg_lr2, m2, w2);
  w0 = w2n.x; w1 = w2n.y;
  m0 = m2.x; m1 = m2.y;
}

// The steps of one device on one pack.  Each step is written stage by stage over all NB Philox
// blocks of the pack - all generator rounds, then all radii, one combined test for the rare
// "u0 next to 1" case, then all angles, then the update - so that the independent chains sit in
// the same straight-line code and the hardware scheduler can interleave them.
// The fp32 arithmetic of a step is written on pairs (sm_100's two-wide fp32 instructions: one
// issue slot, two IEEE results, so every value is bit for bit what the scalar form gives): the two
// radii of a block, its two angles, the two normals of a Box-Muller pair and their two parameters.
// The launch is bound by the issue slot with several steps per device, and this takes 22 of 155
// warp instructions out of a step of an 8-parameter pack (measured: K1 -3 ... -4 %, fused round
// -4 ... -5 %).
template <typename Gen, int NB>
__device__ __forceinline__ void sgd_steps(float (&w)[4 * NB], float (&m)[4 * NB],
                                          const GroupProducts<NB> &gp, const RowStep &rs,
                                          const PhiloxKeys &keys, const StepConsts &k) {
  uint32_t c2_first[NB];
#pragma unroll
  for (int b = 0; b < NB; ++b) c2_first[b] = gp.hi[b] ^ rs.r1_c2;
  const float2 wd2 = make_float2(k.wd, k.wd), mu2 = make_float2(k.mu, k.mu);
  const float2 neg_lr2 = make_float2(k.neg_lr, k.neg_lr);
  for (int e = 0; e < rs.steps; ++e) {
    const uint32_t c0_first = rs.r1_c0 ^ (rs.base_lo + (uint32_t)e);
    uint32_t x[NB][4];
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      x[b][0] = c0_first; x[b][1] = rs.r1_c1; x[b][2] = c2_first[b]; x[b][3] = gp.lo[b];
    }
#pragma unroll
    for (int r = 1; r < 10; ++r)
#pragma unroll
      for (int b = 0; b < NB; ++b) philox_round(x[b][0], x[b][1], x[b][2], x[b][3], keys.a[r], keys.b[r]);
    float2 r2[NB];  // squared radii of the block's two pairs
    uint32_t top = 0;
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      r2[b] = Gen::radius2_pair(x[b][0], x[b][2], k.lg_scale);
      top = max(top, max(x[b][0], x[b][2]));
    }
    if (Gen::needs_series(top)) {  // about once in 250 steps of a pack
#pragma unroll
      for (int b = 0; b < NB; ++b) {
        if (Gen::needs_series(x[b][0])) r2[b].x = r2_next_to_one(x[b][0], k.scale2);
        if (Gen::needs_series(x[b][2])) r2[b].y = r2_next_to_one(x[b][2], k.scale2);
      }
    }
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      const float2 theta = Gen::angle_pair(x[b][1], x[b][3]);
      const float2 n01 = Gen::finish_pair(r2[b].x, theta.x);  // grad_std * (z0, z1)
      const float2 n23 = Gen::finish_pair(r2[b].y, theta.y);  // grad_std * (z2, z3)
      sgd_update_pair(w[4 * b], w[4 * b + 1], m[4 * b], m[4 * b + 1], n01, wd2, mu2, neg_lr2);
      sgd_update_pair(w[4 * b + 2], w[4 * b + 3], m[4 * b + 2], m[4 * b + 3], n23, wd2, mu2, neg_lr2);
    }
  }
}

// ------------------------------------------------------------------------------------------
// Reduced-precision state (a workload variant outside the paper, which trains in fp32): the one
// rounding to bf16 at the end of a local-update call may be stochastic.  The 16 random bits are
// added to the fp32 bit pattern below the bf16 mantissa and the sum is truncated: a finite value
// moves to its neighbour of larger magnitude with probability (discarded bits) / 2^16, so the
// expectation is the value itself.  Infinities and NaNs are rounded to nearest even.
// The bits come from one Philox block per column group and call, counter
// (group, index of the call's last step, device, 'R' << 24 | index >> 32): element `lane` of the
// group takes the low half of word `lane` for its parameter and the high half for its momentum.
// The result is exactly representable in bf16, so the conversion at the store changes nothing.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ float bf16_stochastic(float v, uint32_t r16) {
  const uint32_t bits = __float_as_uint(v);
  if ((bits & 0x7F800000u) == 0x7F800000u) return __bfloat162float(__float2bfloat16_rn(v));
  return __uint_as_float((bits + r16) & 0xFFFF0000u);
}

template <typename MT, int NB>
__device__ __forceinline__ void round_stochastic(float (&w)[4 * NB], float (&m)[4 * NB], int64_t pack,
                                                 const RowStep &rs, const PhiloxKeys &keys) {
#pragma unroll
  for (int b = 0; b < NB; ++b) {
    uint32_t x0 = (uint32_t)(pack * NB + b);
    uint32_t x1 = rs.base_lo + (uint32_t)rs.steps - 1u;
    uint32_t x2 = (uint32_t)rs.row;
    uint32_t x3 = rs.r1_c2 ^ keys.b[0] ^ (kTagGrad ^ kTagRound);  // tag | high bits of the step index
    philox4x32_10(x0, x1, x2, x3, keys);
    const uint32_t x[4] = {x0, x1, x2, x3};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      w[4 * b + i] = bf16_stochastic(w[4 * b + i], x[i] & 0xFFFFu);
      if (sizeof(MT) == 2) m[4 * b + i] = bf16_stochastic(m[4 * b + i], x[i] >> 16);
    }
  }
}

// Row addressing: the host passes each row's byte offset, the thread adds the byte offset of its
// pack once, so a row access costs one 64-bit add.
template <typename WT>
__device__ __forceinline__ WT *at_row(char *pack_in_row0, int64_t row_off) {
  return reinterpret_cast<WT *>(pack_in_row0 + row_off);
}

// WT / MT: storage types of the parameters and of the momentum (bf16 momentum only with bf16
// parameters); RM = 1: the bf16 stores of this call are rounded stochastically.
template <typename WT, typename MT, typename Gen, int E, int RM>
__global__ void __launch_bounds__(kThreads)
k_local_step(WT *__restrict__ w, MT *__restrict__ m, int64_t n_params, LocalStepArgs a,
             PhiloxKeys keys, StepConsts k) {
  const int64_t p = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  // The body is compiled twice: for blocks whose packs are all full (`live` is then the constant
  // E and every ragged-tail test in the loads and stores folds away: 2-3 % fewer instructions per
  // row) and for the one block that holds the end of the vector.
  auto run = [&](auto all_full) {
    const int live = decltype(all_full)::value ? E : live_of(n_params, p, E);
    if (live == 0) return;
    const GroupProducts<E / 4> gp(p);
    char *wp = reinterpret_cast<char *>(w) + p * (int64_t)(E * sizeof(WT));
    char *mp = reinterpret_cast<char *>(m) + p * (int64_t)(E * sizeof(MT));

    auto load = [&](int j, RawPack<WT, E> &rw, RawPack<MT, E> &rm) {
      ld_raw(at_row<WT>(wp, a.r[j].w_off), live, rw);
      ld_raw(at_row<MT>(mp, a.r[j].m_off), live, rm);
    };
    auto body = [&](int j, float (&wv)[E], float (&mv)[E]) {
      sgd_steps<Gen, E / 4>(wv, mv, gp, a.r[j], keys, k);
      if constexpr (RM == 1) round_stochastic<MT, E / 4>(wv, mv, p, a.r[j], keys);
      st_pack_any(at_row<WT>(wp, a.r[j].w_off), 0, live, wv);
      st_pack_any(at_row<MT>(mp, a.r[j].m_off), 0, live, mv);
    };
    // fp32 values are updated in the registers they were loaded into; bf16 ones are widened first
    auto visit = [&](int j, RawPack<WT, E> &rw, RawPack<MT, E> &rm) {
      if constexpr (sizeof(WT) == 4) {
        body(j, rw.v, rm.v);
      } else if constexpr (sizeof(MT) == 4) {
        float wv[E];
        unpack(rw, wv);
        body(j, wv, rm.v);
      } else {
        float wv[E], mv[E];
        unpack(rw, wv);
        unpack(rm, mv);
        body(j, wv, mv);
      }
    };
    // No prefetch of the next row: the registers it would take cost a resident block, and four
    // blocks per SM hide the row loads better than three blocks with a prefetch (measured).
    // Grid: x = chunks of kThreads packs; y = 1: the block walks over all listed rows (every thread
    // mixes light and heavy rows, so memory-bound and arithmetic-bound phases overlap), or
    // y = number of rows: one row per block (eight times more, shorter blocks: no partial last
    // wave, which is worth 5-7 % when every row is memory-bound).  The host chooses.
    RawPack<WT, E> rw;
    RawPack<MT, E> rm;
    const int j_begin = gridDim.y > 1 ? (int)blockIdx.y : 0;
    const int j_end = gridDim.y > 1 ? j_begin + 1 : a.n;
    for (int j = j_begin; j < j_end; ++j) {
      load(j, rw, rm);
      visit(j, rw, rm);
    }
  };
  if (((int64_t)blockIdx.x + 1) * kThreads * E <= n_params)
    run(std::true_type{});
  else
    run(std::false_type{});
}

// ------------------------------------------------------------------------------------------
// K2: fused weighted combination of `nr` rows written to `nw` rows in the same pass.
//   partial aggregation (Eq. 5): read list = write list = the selected devices, weights a_j;
//   global synchronisation (Algorithm 1): read list = {source}, weight 1, write list = receivers.
//   acc = a_0 * w[rd_0];  acc = fma(a_j, w[rd_j], acc) for j = 1 .. nr-1, in list order.
// A thread owns U 16-byte packs.  KR > 0: compile-time read count; KR == 0: any read count.  The
// row loads of a pack are issued in batches of B rows (B * E values in registers) before the
// batch's multiply-adds; U packs per thread keep enough bytes in flight when the list is short.
// ------------------------------------------------------------------------------------------
struct CombineArgs {
  int32_t nr;
  int32_t nw;
  int32_t rd[kMaxDevices];
  float a[kMaxDevices];
  int32_t wr[kMaxDevices];
};

template <typename WT, int KR, int E>
__device__ __forceinline__ void combine_pack(const WT *__restrict__ w, int64_t stride,
                                             const CombineArgs &c, int64_t p, int live,
                                             float (&acc)[E]) {
  constexpr int B = KR > 0 ? (KR <= 16 ? KR : 16) : 8;  // rows per batch: at most 16 x 16 bytes in registers
  const int nr = KR > 0 ? KR : c.nr;
#pragma unroll
  for (int i = 0; i < E; ++i) acc[i] = 0.f;
#pragma unroll
  for (int base = 0; base < (KR > 0 ? KR : kMaxDevices); base += B) {
    if (base >= nr) break;
    RawPack<WT, E> raw[B];
#pragma unroll
    for (int j = 0; j < B; ++j)
      if (base + j < nr) ld_raw(w + (int64_t)c.rd[base + j] * stride + (int64_t)E * p, live, raw[j]);
#pragma unroll
    for (int j = 0; j < B; ++j) {
      if (base + j < nr) {
        const float aj = c.a[base + j];
        float v[E];
        unpack(raw[j], v);
        if (base + j == 0) {
#pragma unroll
          for (int i = 0; i < E; ++i) acc[i] = __fmul_rn(aj, v[i]);
        } else {
#pragma unroll
          for (int i = 0; i < E; ++i) acc[i] = fmaf(aj, v[i], acc[i]);
        }
      }
    }
  }
}

template <typename WT, int KR, int U>
__global__ void __launch_bounds__(kThreads)
k_combine(WT *__restrict__ w, int64_t stride, int64_t n_params, CombineArgs c) {
  constexpr int E = Pack16<WT>::E;
  // Blocks walk the vector from its END to its start: the local update before it in a round walks
  // it from the start, so what that kernel left in the 126 MB L2 - the end of every row - is read
  // first.  Measured inside a round on the ResNet-18-sized workload (k = 4): 159 of the 179 MB of
  // reads come from DRAM instead of all of them, 61 -> 57 us.
  const int64_t chunk = (int64_t)(gridDim.x - 1 - blockIdx.x);
  const int64_t p0 = chunk * (kThreads * U) + threadIdx.x;
  // Fast path (all but the last chunk of a launch): every pack of the block is full, so the
  // U * KR row loads of a thread are straight-line code and all in flight together.
  const bool block_full = ((chunk + 1) * (kThreads * U)) * E <= n_params;
  if (KR > 0 && KR * U <= 16 && block_full) {
    constexpr int KRc = KR > 0 ? KR : 1;
    RawPack<WT, E> raw[U][KRc];
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int j = 0; j < KRc; ++j)
        ld_raw(w + (int64_t)c.rd[j] * stride + (int64_t)E * (p0 + (int64_t)u * kThreads), E, raw[u][j]);
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float acc[E], v[E];
      unpack(raw[u][0], v);
#pragma unroll
      for (int i = 0; i < E; ++i) acc[i] = __fmul_rn(c.a[0], v[i]);
#pragma unroll
      for (int j = 1; j < KRc; ++j) {
        unpack(raw[u][j], v);
#pragma unroll
        for (int i = 0; i < E; ++i) acc[i] = fmaf(c.a[j], v[i], acc[i]);
      }
      for (int j = 0; j < c.nw; ++j)
        st_pack<E>(w + (int64_t)c.wr[j] * stride, p0 + (int64_t)u * kThreads, acc);
    }
    return;
  }
  float acc[U][E];
  int live[U];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const int64_t p = p0 + (int64_t)u * kThreads;
    live[u] = live_of(n_params, p, E);
    if (live[u] > 0) combine_pack<WT, KR, E>(w, stride, c, p, live[u], acc[u]);
  }
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const int64_t p = p0 + (int64_t)u * kThreads;
    if (live[u] > 0)
      for (int j = 0; j < c.nw; ++j) st_pack_any(w + (int64_t)c.wr[j] * stride, p, live[u], acc[u]);
  }
}

// ------------------------------------------------------------------------------------------
// Integration of a received model (Section "Model aggregation and fault-tolerant": an unselected
// device folds the received parameters into its own; read here as a convex combination, beside the
// overwrite that k_combine provides):
//   w[dst_j] = fma(beta, w[src], (1 - beta) * w[dst_j])   for every receiver j,
// the product rounded to fp32 before the fused multiply-add.  A thread owns U 16-byte packs; per
// pack the sender's values are loaded once and the receivers' rows are loaded in batches of 8
// before the batch's arithmetic and stores.  1 + n reads and n writes per element.
// ------------------------------------------------------------------------------------------
struct MixArgs {
  int32_t n;    // receivers
  int32_t src;  // sender
  float beta, one_minus_beta;
  int32_t dst[kMaxDevices];
};

template <typename WT, int U>
__global__ void __launch_bounds__(kThreads)
k_integrate(WT *__restrict__ w, int64_t stride, int64_t n_params, MixArgs a) {
  constexpr int E = Pack16<WT>::E;
  constexpr int B = 8;
  const int64_t p0 = (int64_t)blockIdx.x * (kThreads * U) + threadIdx.x;
  int live[U];
  RawPack<WT, E> from[U];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const int64_t p = p0 + (int64_t)u * kThreads;
    live[u] = live_of(n_params, p, E);
    if (live[u] > 0) ld_raw(w + (int64_t)a.src * stride + (int64_t)E * p, live[u], from[u]);
  }
#pragma unroll
  for (int u = 0; u < U; ++u) {
    if (live[u] == 0) continue;
    const int64_t p = p0 + (int64_t)u * kThreads;
    float s[E];
    unpack(from[u], s);
    for (int base = 0; base < a.n; base += B) {
      RawPack<WT, E> raw[B];
#pragma unroll
      for (int j = 0; j < B; ++j)
        if (base + j < a.n) ld_raw(w + (int64_t)a.dst[base + j] * stride + (int64_t)E * p, live[u], raw[j]);
#pragma unroll
      for (int j = 0; j < B; ++j) {
        if (base + j < a.n) {
          float v[E];
          unpack(raw[j], v);
#pragma unroll
          for (int i = 0; i < E; ++i) v[i] = fmaf(a.beta, s[i], __fmul_rn(a.one_minus_beta, v[i]));
          st_pack_any(w + (int64_t)a.dst[base + j] * stride, p, live[u], v);
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// Deterministic reductions shared by the statistics kernel and the fused round kernel.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
  return v;
}

// Last-block finish: the block that draws the last ticket sums partials[t][0 .. n_src) for every
// t < n_vals in a fixed order (a warp per value, lanes strided, then the butterfly), hands the
// sums to `emit`, and resets the ticket.  Returns without waiting for anyone.
template <typename Emit>
__device__ __forceinline__ void finish_by_last_block(const double *__restrict__ partials,
                                                     int n_vals, int n_src,
                                                     unsigned int *__restrict__ ticket,
                                                     bool *s_last, Emit emit) {
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) *s_last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
  __syncthreads();
  if (!*s_last) return;
  __threadfence();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int t = warp; t < n_vals; t += kThreads / 32) {
    const double *src = partials + (int64_t)t * n_src;
    double s = 0.0;
    for (int l = lane; l < n_src; l += 32) s += __ldcg(src + l);
    s = warp_sum(s);
    if (lane == 0) emit(t, s);
  }
  if (threadIdx.x == 0) *ticket = 0u;
}

// Two-level variant for grids of many blocks (the fused round).  Blocks are grouped in runs of
// kFinishGroup consecutive block indices.  The block that draws a group's last ticket sums that
// group's partials[t][first block of the group ...] in block order -> group_partials[t][group]
// and draws the launch's ticket; the block that draws the last of those sums the group sums in
// group order and hands them to `emit`.  Each of the two sums has a fixed order that does not
// depend on which block happens to compute it, so the result is reproducible; no block waits for
// another; all tickets are back at zero when the launch ends.
constexpr int kFinishGroup = 128;

template <typename Emit>
__device__ __forceinline__ void finish_two_level(const double *__restrict__ partials,
                                                 double *__restrict__ group_partials, int n_vals,
                                                 unsigned int *__restrict__ group_tickets,
                                                 unsigned int *__restrict__ ticket, bool *s_last,
                                                 Emit emit) {
  const int n_blocks = (int)gridDim.x;
  const int n_groups = (n_blocks + kFinishGroup - 1) / kFinishGroup;
  const int g = (int)blockIdx.x / kFinishGroup;
  const int g_first = g * kFinishGroup;
  const int g_size = min(kFinishGroup, n_blocks - g_first);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) *s_last = (atomicAdd(group_tickets + g, 1u) == (unsigned)g_size - 1u);
  __syncthreads();
  if (!*s_last) return;
  __threadfence();
  for (int t = warp; t < n_vals; t += kThreads / 32) {
    const double *src = partials + (int64_t)t * n_blocks + g_first;
    double s = 0.0;
    for (int l = lane; l < g_size; l += 32) s += __ldcg(src + l);
    s = warp_sum(s);
    if (lane == 0) {
      if (n_groups == 1) {  // a single group: its sum is the result (the second level would add 0 to it)
        emit(t, s);
      } else if (access_ok(group_partials + (int64_t)t * n_groups + g, 8)) {
        group_partials[(int64_t)t * n_groups + g] = s;
      }
    }
  }
  if (n_groups == 1) {
    if (threadIdx.x == 0) group_tickets[g] = 0u;
    return;
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    group_tickets[g] = 0u;
    *s_last = (atomicAdd(ticket, 1u) == (unsigned)n_groups - 1u);
  }
  __syncthreads();
  if (!*s_last) return;
  __threadfence();
  for (int t = warp; t < n_vals; t += kThreads / 32) {
    const double *src = group_partials + (int64_t)t * n_groups;
    double s = 0.0;
    for (int l = lane; l < n_groups; l += 32) s += __ldcg(src + l);
    s = warp_sum(s);
    if (lane == 0) emit(t, s);
  }
  if (threadIdx.x == 0) *ticket = 0u;
}

// ------------------------------------------------------------------------------------------
// K3: per-replica squared norm and squared distance to a reference replica.
// Block b works on row b % N and on the chunks (b / N), (b / N) + lanes, ...; a chunk is
// kThreads * U 16-byte packs.  Blocks that are neighbours in launch order work on the same chunk
// of different rows at about the same time, so the reference chunk is fetched from HBM once and
// found in L2 by the others: HBM traffic stays N * P elements.
// Per thread: fp32 sums over the elements of a chunk in a fixed order, accumulated in fp64 across
// chunks; butterfly over the warp and a fixed-order sum over the warps (fp64) give
// partials[which * N + row][lane].  The last-ticket block sums them -> out[2N] (norm2 then div2).
// No block waits for another; fixed grid and fixed orders make the result reproducible.
// ------------------------------------------------------------------------------------------
template <typename WT, int U>
__global__ void __launch_bounds__(kThreads)
k_stats(const WT *__restrict__ w, int64_t stride, int64_t n_params, int n_devices, int ref,
        int lanes, double *__restrict__ partials, unsigned int *__restrict__ ticket,
        float *__restrict__ out) {
  constexpr int kWarps = kThreads / 32;
  constexpr int E = Pack16<WT>::E;
  __shared__ double s_part[2][kWarps];
  __shared__ bool s_last;
  const int row = blockIdx.x % n_devices;
  const int my_lane = blockIdx.x / n_devices;
  const int64_t n_packs = (n_params + E - 1) / E;
  const int64_t per_chunk = (int64_t)kThreads * U;
  const int64_t n_chunks = (n_packs + per_chunk - 1) / per_chunk;
  const WT *my_row = w + (int64_t)row * stride;
  const WT *ref_row = w + (int64_t)ref * stride;

  double n2 = 0.0, d2 = 0.0;
  for (int64_t chunk = my_lane; chunk < n_chunks; chunk += lanes) {
    const int64_t p0 = chunk * per_chunk + threadIdx.x;
    RawPack<WT, E> rv[U], rr[U];
    if ((chunk + 1) * per_chunk * E <= n_params) {  // every pack of the chunk is full: no branches
#pragma unroll
      for (int u = 0; u < U; ++u) {
        ld_raw(my_row + (int64_t)E * (p0 + (int64_t)u * kThreads), E, rv[u]);
        ld_raw(ref_row + (int64_t)E * (p0 + (int64_t)u * kThreads), E, rr[u]);
      }
    } else {
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int64_t p = p0 + (int64_t)u * kThreads;
        const int live = live_of(n_params, p, E);
        if (live > 0) {
          ld_raw(my_row + (int64_t)E * p, live, rv[u]);
          ld_raw(ref_row + (int64_t)E * p, live, rr[u]);
        } else {
          zero_raw(rv[u]);
          zero_raw(rr[u]);
        }
      }
    }
    float a = 0.f, b = 0.f;
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float v[E], r[E];
      unpack(rv[u], v);
      unpack(rr[u], r);
#pragma unroll
      for (int i = 0; i < E; ++i) {
        const float d = v[i] - r[i];
        a = fmaf(v[i], v[i], a);
        b = fmaf(d, d, b);
      }
    }
    n2 += (double)a;
    d2 += (double)b;
  }
  n2 = warp_sum(n2);
  d2 = warp_sum(d2);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) {
    s_part[0][warp] = n2;
    s_part[1][warp] = d2;
  }
  __syncthreads();
  if (threadIdx.x < 2) {
    double s = 0.0;
    for (int wi = 0; wi < kWarps; ++wi) s += s_part[threadIdx.x][wi];
    double *slot = partials + ((int64_t)threadIdx.x * n_devices + row) * lanes + my_lane;
    if (access_ok(slot, 8)) *slot = s;
  }
  finish_by_last_block(partials, 2 * n_devices, lanes, ticket, &s_last,
                       [&](int t, double sum) {
                         if (access_ok(out + t, 4)) out[t] = (float)sum;
                       });
}

// ------------------------------------------------------------------------------------------
// Fused round: local update of every device, partial aggregation with write-back (optionally
// sent to every device: global synchronisation) and the statistics, in ONE pass over the arena.
// Selection only needs the versions, which the host knows before the steps run, so the selected
// set is an input.  Per pack a thread visits the rows in the order "selected devices in draw
// order, then the others": it runs each row's steps in registers exactly as K1 does, folds the
// selected rows into the aggregate in draw order exactly as K2 does (acc = a_0 w_0, then fma),
// writes the aggregate to the selected rows when the last of them is done, and for every row adds
// the squares of what the row now holds, and of its distance to the aggregate, to the row's sums.
// Parameters and momentum come out bit-identical to K1 followed by K2 (and the broadcast); the
// aggregate is never re-read from memory, so a round moves 16 bytes per (device, parameter)
// instead of 20 + 8k/N.
//
// Grid: one block per chunk of kThreads packs, up to a cap beyond which the blocks stride over
// the chunks; the hardware block scheduler then balances the SMs (a one-wave persistent grid ends
// with a partly filled last pass and keeps all blocks in the same phase of their rows: measured
// 7-15 % slower with several steps per device).  The chunk loop's trip count depends on the block
// index only, so control flow and every row descriptor read inside it are uniform across the
// block - with a per-thread loop bound the compiler re-read the descriptors through indexed
// constant loads in every step (+7 instructions per step).  Lanes beyond the end of the vector
// (live = 0) take part in everything: their loads return zeros, their stores store nothing, and
// what they compute is zeroed before it is summed.
// Row sums: one shuffle per row and pack, then a shared-memory slot owned by the thread (fp32); at
// the end of a chunk's round, per row, a fixed-order sum over the warps and a butterfly over each
// half-warp (fp64), added to the block's sums of that round; at the end of the block
// partials[round][value][block] and a two-level last-ticket finish per round.  Deterministic.
// Dynamic shared memory: n * kThreads floats.  64 registers: four resident blocks per SM.
// NR > 1: the launch takes a batch of up to NR consecutive rounds.  A block carries its chunk
// through all of them before it moves on (chunk loop outside, round loop inside), so from the
// second round on the rows come from L2 and not from HBM, and every round still leaves its own
// statistics.  Results are those of the rounds launched one by one, bit for bit.
// E = 4 (fp32 only): packs of 4 columns, one Philox block per thread.  A block then holds half
// the rows at a time, which keeps the rows of all resident blocks within the L2 for up to about
// 20 devices: the form batches of one-step rounds take (the host decides).  Statistics are then
// folded over chunks of 1024 columns: equal to the other forms to rounding, not bit for bit.
// PF = true is a second build that issues the next row's loads before the current row's steps
// (80 registers, three resident blocks).  With bf16 parameters a row is 48 bytes per thread or
// less, and when every device runs one or two steps the launch is bound by how many bytes are in
// flight: the prefetch is worth 6-8 % there (and costs 1-3 % with more steps, and 0-13 % with fp32
// parameters at any step count), so the host takes it for exactly that case.
// ------------------------------------------------------------------------------------------
struct RoundArgs {
  int32_t n;          // rows visited = all N devices: [0, k) selected in draw order, then the rest
  int32_t k;          // number of selected devices, 1 <= k <= n
  int32_t write_all;  // global synchronisation: 0 none, 1 every other device receives the aggregate
                      // (overwrite), 2 every other device mixes it into its own model
  float beta, one_minus_beta;  // weights of the mix (write_all = 2), as in k_integrate
  float a[kMaxDevices];  // aggregation weights of the selected devices
  RowStep r[kMaxDevices];
};

// Adds a thread's (sum of squares, sum of squared distances) for one row to the block's
// accumulators.  One shuffle folds lane l and lane l ^ 16 so that the lower half-warp carries the
// first value and the upper half the second; each thread then owns ONE fp32 slot per row,
// s_acc[visit index][thread], which it alone updates (no atomics, fixed order).
__device__ __forceinline__ void add_row_sums(float *s_acc, int j, float n2, float d2, int lane) {
  const bool upper = (lane & 16) != 0;
  const float keep = upper ? d2 : n2;
  const float give = upper ? n2 : d2;
  float *slot = s_acc + j * kThreads + threadIdx.x;
  *slot += keep + __shfl_xor_sync(0xFFFFFFFFu, give, 16);
}

constexpr int kRoundBlocksPerSM = 4;

// A batch of consecutive rounds for one launch.  Every operation of a round is elementwise in the
// parameter index and the selections are known to the host beforehand, so a thread can take its
// pack through several rounds back to back: what it wrote in one round it reads back in the next
// (the same thread, the same addresses, program order), while the lines are still in L2.
template <int NR>
struct RoundBatch {
  int32_t n_rounds;  // 1 <= n_rounds <= NR
  RoundArgs round[NR];
};
constexpr int kRoundBatchMax = 8;

// Scratch of the fused round kernel, per round of a batch.
struct RoundScratch {
  double *partials;            // [round][2 n][blocks]
  double *group_partials;      // [round][2 n][groups]
  unsigned int *tickets;       // [round][1 + groups]: the round's ticket, then one per group
  float *out_rounds;           // [round][2 kMaxDevices]: the statistics of every round of the batch
  float *out;                  // [2 kMaxDevices]: the statistics of the batch's last round
};

template <typename WT, typename MT, typename Gen, int E, int RM, bool PF, int NR>
__global__ void __launch_bounds__(kThreads, PF ? kRoundBlocksPerSM - 1 : kRoundBlocksPerSM)
k_round(WT *__restrict__ w, MT *__restrict__ m, int64_t n_params, RoundBatch<NR> b, PhiloxKeys keys,
        StepConsts k, RoundScratch scratch) {
  constexpr int kWarps = kThreads / 32;
  extern __shared__ float s_acc[];  // [n][kThreads]: per-thread row sums of the round in hand
  __shared__ double s_part[NR][2 * kMaxDevices];  // the block's sums, per round
  __shared__ bool s_last;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n_dev = b.round[0].n;
  for (int j = 0; j < n_dev; ++j) s_acc[j * kThreads + threadIdx.x] = 0.f;
  for (int t = threadIdx.x; t < NR * 2 * kMaxDevices; t += kThreads) (&s_part[0][0])[t] = 0.0;
  __syncthreads();

  const int64_t n_packs = (n_params + E - 1) / E;
  const int64_t n_chunks = (n_packs + kThreads - 1) / kThreads;
  for (int64_t chunk = blockIdx.x; chunk < n_chunks; chunk += gridDim.x) {
    // The chunk's work is compiled twice: for chunks whose packs are all full (`live` is then the
    // constant E and every ragged-tail test in the loads and stores folds away) and for the chunk
    // that holds the end of the vector (and, there, the lanes beyond it).
    auto do_chunk = [&](auto all_full) {
      const int64_t p = chunk * kThreads + threadIdx.x;
      const int live = decltype(all_full)::value ? E : live_of(n_params, p, E);
      const GroupProducts<E / 4> gp(p);
      char *wp = reinterpret_cast<char *>(w) + p * (int64_t)(E * sizeof(WT));
      char *mp = reinterpret_cast<char *>(m) + p * (int64_t)(E * sizeof(MT));

      auto do_round = [&](const RoundArgs &a, const int r) {
        // Row j as it is after its local steps: loads w (and m when the row runs steps), runs the
        // steps, stores the momentum, and leaves in wv what the row now holds (as stored; dead lanes
        // 0).  fp32 values are updated in the registers they were loaded into.
        // PF: the next row's loads are issued before this row's steps (see the kernel's header).
        RawPack<WT, E> rw_next;
        RawPack<MT, E> rm_next;
        auto fetch = [&](int j) {
          ld_raw(at_row<WT>(wp, a.r[j].w_off), live, rw_next);
          if (a.r[j].steps > 0) ld_raw(at_row<MT>(mp, a.r[j].m_off), live, rm_next);
        };
        if constexpr (PF) fetch(0);
        auto row_after_steps = [&](int j, float (&wv)[E]) -> bool {
          RawPack<WT, E> rw;
          RawPack<MT, E> rm;
          if constexpr (PF) {
            rw = rw_next;
            rm = rm_next;
            if (j + 1 < a.n) fetch(j + 1);
          } else {
            ld_raw(at_row<WT>(wp, a.r[j].w_off), live, rw);
          }
          const bool stepped = a.r[j].steps > 0;
          if (stepped) {
            if constexpr (!PF) ld_raw(at_row<MT>(mp, a.r[j].m_off), live, rm);
            float mv[E];
            unpack(rw, wv);
            unpack(rm, mv);
            sgd_steps<Gen, E / 4>(wv, mv, gp, a.r[j], keys, k);
            if constexpr (RM == 1) round_stochastic<MT, E / 4>(wv, mv, p, a.r[j], keys);
            st_pack_any(at_row<MT>(mp, a.r[j].m_off), 0, live, mv);
#pragma unroll
            for (int i = 0; i < E; ++i) wv[i] = as_stored(wv[i], w);
            if (live < E) {  // the ragged last pack of a row and the lanes beyond it: dead lanes stay 0
#pragma unroll
              for (int i = 0; i < E; ++i) wv[i] = i < live ? wv[i] : 0.f;
            }
          } else {
            unpack(rw, wv);
          }
          return stepped;
        };

        // ---- the selected devices in draw order: acc = a_0 w_0, then acc = fma(a_j, w_j, acc)
        float acc[E];
        {
          float wv[E];
          row_after_steps(0, wv);
          const float a0 = a.a[0];
#pragma unroll
          for (int i = 0; i < E; ++i) acc[i] = __fmul_rn(a0, wv[i]);
        }
        for (int j = 1; j < a.k; ++j) {
          float wv[E];
          row_after_steps(j, wv);
          const float aj = a.a[j];
#pragma unroll
          for (int i = 0; i < E; ++i) acc[i] = fmaf(aj, wv[i], acc[i]);
        }
        {
          float n2 = 0.f;
#pragma unroll
          for (int i = 0; i < E; ++i) {
            acc[i] = as_stored(acc[i], w);
            n2 = fmaf(acc[i], acc[i], n2);
          }
          // a single selected device that ran no steps already holds the aggregate (a_0 = 1)
          if (a.k > 1 || a.r[0].steps > 0)
            for (int t = 0; t < a.k; ++t) st_pack_any(at_row<WT>(wp, a.r[t].w_off), 0, live, acc);
          add_row_sums(s_acc, a.k - 1, n2, 0.f, lane);  // one value for all selected devices
        }
        // ---- the other devices: keep their own model, or receive the aggregate
        for (int j = a.k; j < a.n; ++j) {
          float wv[E];
          const bool stepped = row_after_steps(j, wv);
          if (a.write_all == 1) {
#pragma unroll
            for (int i = 0; i < E; ++i) wv[i] = acc[i];
          } else if (a.write_all == 2) {
#pragma unroll
            for (int i = 0; i < E; ++i)
              wv[i] = as_stored(fmaf(a.beta, acc[i], __fmul_rn(a.one_minus_beta, wv[i])), w);
          }
          if (stepped || a.write_all) st_pack_any(at_row<WT>(wp, a.r[j].w_off), 0, live, wv);
          float n2 = 0.f, d2 = 0.f;
#pragma unroll
          for (int i = 0; i < E; ++i) {
            const float d = wv[i] - acc[i];
            n2 = fmaf(wv[i], wv[i], n2);
            d2 = fmaf(d, d, d2);
          }
          add_row_sums(s_acc, j, n2, d2, lane);
        }
        // ---- block: fold the per-thread slots of every visit index j >= k - 1 into the block's
        // sums of this round and clear them.  Warp w takes the visit indices k - 1 + w,
        // k - 1 + w + 8, ...: each lane adds the slots of the threads that share its lane index
        // (one per warp, in warp order; lower half-warps hold norms, upper halves distances), then a
        // butterfly over the half-warp finishes the two sums.
        __syncthreads();
        for (int j = a.k - 1 + warp; j < a.n; j += kWarps) {
          float v = 0.f;
#pragma unroll
          for (int wi = 0; wi < kWarps; ++wi) {
            v += s_acc[j * kThreads + wi * 32 + lane];
            s_acc[j * kThreads + wi * 32 + lane] = 0.f;
          }
          double d = (double)v;
#pragma unroll
          for (int off = 8; off > 0; off >>= 1) d += __shfl_xor_sync(0xFFFFFFFFu, d, off);
          if ((lane & 15) == 0) s_part[r][2 * j + (lane >> 4)] += d;  // value = 2 * visit index + which
        }
        __syncthreads();
      };
      // A launch of a single round reads its arguments at constant addresses (the compiler then
      // keeps the row descriptors on the uniform datapath); a batch indexes them by the round.
      if constexpr (NR == 1) {
        do_round(b.round[0], 0);
      } else {
        for (int r = 0; r < b.n_rounds; ++r) do_round(b.round[r], r);
      }
    };
    if ((chunk + 1) * kThreads * E <= n_params)
      do_chunk(std::true_type{});
    else
      do_chunk(std::false_type{});
  }
  // ---- launch: per round, partials[value][block] and the two-level last-ticket finish
  const int n_blocks = (int)gridDim.x;
  const int n_groups = (n_blocks + kFinishGroup - 1) / kFinishGroup;
  for (int r = 0; r < (NR == 1 ? 1 : b.n_rounds); ++r) {
    const RoundArgs &a = b.round[NR == 1 ? 0 : r];
    const int ksel = a.k;
    double *partials = scratch.partials + (int64_t)r * 2 * n_dev * n_blocks;
    double *group_partials = scratch.group_partials + (int64_t)r * 2 * n_dev * n_groups;
    unsigned int *tickets = scratch.tickets + (int64_t)r * (1 + n_groups);
    float *out_r = scratch.out_rounds + r * 2 * kMaxDevices;
    const bool is_last_round = r + 1 == (NR == 1 ? 1 : b.n_rounds);
    auto put = [&](int at, float v) {  // every round's statistics; the last round's also where hadfl_stats puts them
      if (access_ok(out_r + at, 4)) out_r[at] = v;
      if (is_last_round && access_ok(scratch.out + at, 4)) scratch.out[at] = v;
    };
    for (int t = 2 * (ksel - 1) + threadIdx.x; t < 2 * n_dev; t += kThreads) {
      double *slot = partials + (int64_t)t * n_blocks + blockIdx.x;
      if (access_ok(slot, 8)) *slot = s_part[r][t];
    }
    finish_two_level(partials + (int64_t)2 * (ksel - 1) * n_blocks,
                     group_partials + (int64_t)2 * (ksel - 1) * n_groups, 2 * (n_dev - ksel + 1),
                     tickets + 1, tickets, &s_last, [&](int t, double sum) {
      const int j = ksel - 1 + (t >> 1), which = t & 1;
      if (j == ksel - 1) {  // the selected devices share one norm and are at distance 0
        for (int q = 0; q < ksel; ++q) put(which * n_dev + a.r[q].row, which ? 0.f : (float)sum);
      } else {
        put(which * n_dev + a.r[j].row, (float)sum);
      }
    });
  }
}

// ------------------------------------------------------------------------------------------
// Generator diagnostics.
// ------------------------------------------------------------------------------------------
__global__ void k_debug_philox(const uint32_t *__restrict__ ctr, PhiloxKeys keys, int64_t n,
                               uint32_t *__restrict__ out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  uint32_t c0 = ctr[4 * i], c1 = ctr[4 * i + 1], c2 = ctr[4 * i + 2], c3 = ctr[4 * i + 3];
  philox4x32_10(c0, c1, c2, c3, keys);
  out[4 * i] = c0; out[4 * i + 1] = c1; out[4 * i + 2] = c2; out[4 * i + 3] = c3;
}

template <typename Gen>
__global__ void k_debug_normals(const uint32_t *__restrict__ groups, int64_t n, uint32_t c1,
                                uint32_t c2, uint32_t c3, PhiloxKeys keys,
                                float4 *__restrict__ out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  out[i] = normals_of_block<Gen>(groups[i], c1, c2, c3, keys);
}

}  // namespace hadfl
