// sm_100a kernels of the HADFL round: initial model (K0), batched heterogeneity-aware local
// update (K1; Eq. 3 / Algorithm 1), fused weighted aggregation with write-back (K2; Eq. 5), and
// per-replica statistics (K3).
//
// All of them stream rows of one [N][stride] arena.  The unit of work is a "column group": four
// consecutive parameters, one 128-bit access for fp32 storage (64-bit for bf16 storage) and one
// Philox block.  In K1 and K2 a thread owns a column group and walks over the rows, so that
//   - accesses of a warp are 512 contiguous bytes per row,
//   - several independent row loads are in flight per thread before the first dependent use,
//   - every thread does the same amount of arithmetic whatever the per-device step counts are
//     (the kernel-level answer to the straggler problem the paper is about), and
//   - the arithmetic order per element is fixed, hence results are reproducible bit for bit.
// None of this is a dense contraction, so there is no tensor-core path: the bound is HBM
// bandwidth, except for K1 with many steps per device, where the integer multiplies of Philox
// and the special-function unit (log2, sqrt, sin, cos) bind.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "philox.cuh"

namespace hadfl {

constexpr int kMaxDevices = 32;
constexpr int kThreads = 256;

// ------------------------------------------------------------------------------------------
// Storage access: a column group of fp32 or bf16 parameters <-> four fp32 registers.
// `live` is the number of lanes of the group that are parameters (4 except in a ragged last
// group); dead lanes read as 0 and are never written.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ float4 ld_group(const float *row, int64_t g) {
  return *reinterpret_cast<const float4 *>(row + 4 * g);
}
__device__ __forceinline__ void st_group(float *row, int64_t g, float4 v) {
  *reinterpret_cast<float4 *>(row + 4 * g) = v;
}
__device__ __forceinline__ float4 ld_group(const __nv_bfloat16 *row, int64_t g) {
  const uint2 raw = *reinterpret_cast<const uint2 *>(row + 4 * g);
  float4 v;
  v.x = __uint_as_float(raw.x << 16);
  v.y = __uint_as_float(raw.x & 0xFFFF0000u);
  v.z = __uint_as_float(raw.y << 16);
  v.w = __uint_as_float(raw.y & 0xFFFF0000u);
  return v;
}
__device__ __forceinline__ void st_group(__nv_bfloat16 *row, int64_t g, float4 v) {
  const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
  const __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 raw;
  raw.x = *reinterpret_cast<const uint32_t *>(&lo);
  raw.y = *reinterpret_cast<const uint32_t *>(&hi);
  *reinterpret_cast<uint2 *>(row + 4 * g) = raw;
}
__device__ __forceinline__ float ld_elem(const float *row, int64_t p) { return row[p]; }
__device__ __forceinline__ float ld_elem(const __nv_bfloat16 *row, int64_t p) {
  return __bfloat162float(row[p]);
}
__device__ __forceinline__ void st_elem(float *row, int64_t p, float v) { row[p] = v; }
__device__ __forceinline__ void st_elem(__nv_bfloat16 *row, int64_t p, float v) {
  row[p] = __float2bfloat16_rn(v);
}

template <typename T>
__device__ __forceinline__ float4 ld_group_ragged(const T *row, int64_t g, int live) {
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (live > 0) v.x = ld_elem(row, 4 * g + 0);
  if (live > 1) v.y = ld_elem(row, 4 * g + 1);
  if (live > 2) v.z = ld_elem(row, 4 * g + 2);
  return v;
}
template <typename T>
__device__ __forceinline__ void st_group_ragged(T *row, int64_t g, int live, float4 v) {
  if (live > 0) st_elem(row, 4 * g + 0, v.x);
  if (live > 1) st_elem(row, 4 * g + 1, v.y);
  if (live > 2) st_elem(row, 4 * g + 2, v.z);
}
template <typename T>
__device__ __forceinline__ float4 ld_any(const T *row, int64_t g, int live) {
  return live == 4 ? ld_group(row, g) : ld_group_ragged(row, g, live);
}
template <typename T>
__device__ __forceinline__ void st_any(T *row, int64_t g, int live, float4 v) {
  if (live == 4)
    st_group(row, g, v);
  else
    st_group_ragged(row, g, live, v);
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
// 2t + t^2 + (2/3) t^3 (the next term, t^4/2, is below 2^-31 relative).  Kept out of line so that
// the common path pays one compare and an untaken branch for it.
__device__ __noinline__ float r2_next_to_one(uint32_t x0, float scale2) {
  const float t = fmaf(__uint2float_rn(~x0), 0x1p-32f, 0x1p-33f);
  return scale2 * (t * fmaf(t, fmaf(t, 0.66666667f, 1.0f), 2.0f));
}

struct NormalsFast {
  // Two normals of standard deviation s from two words; the caller passes lg_scale = -2 ln2 s^2
  // and scale2 = s^2 so that the scaling costs no instruction:
  //   r^2 = lg_scale * lg2(u0)            (u0 = (x0 + 0.5) 2^-32)
  //   theta = 2 pi a,  a = ((int)x1 + 0.5) 2^-32          (one fused multiply-add)
  // Next to u0 = 1 (x0 >= 2^32 - 2^22) lg2.approx only has an absolute error bound, so the exact
  // complement and a series take over.  Measured against a double-precision evaluation (s = 1):
  // max |dz| about 2e-6, mean 1.6e-7.
  static __device__ __forceinline__ void pair(uint32_t x0, uint32_t x1, float lg_scale,
                                              float scale2, float &z0, float &z1) {
    const float u0 = fmaf(__uint2float_rn(x0), 0x1p-32f, 0x1p-33f);
    float r2 = lg_scale * sfu_lg2(u0);
    if (x0 >= 0xFFC00000u) r2 = r2_next_to_one(x0, scale2);
    const float theta = fmaf(__int2float_rn((int)x1), 1.4629180792671596e-9f, 7.314590396335798e-10f);
    const float r = sfu_sqrt(r2);
    z0 = r * sfu_cos(theta);
    z1 = r * sfu_sin(theta);
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
};

constexpr float kMinusTwoLn2 = -1.3862943611198906f;

// Unit normals of one Philox block.
template <typename Gen>
__device__ __forceinline__ float4 normals_of_block(uint32_t c0, uint32_t c1, uint32_t c2,
                                                   uint32_t c3, const PhiloxKeys &keys) {
  philox4x32_10(c0, c1, c2, c3, keys);
  float4 z;
  Gen::pair(c0, c1, kMinusTwoLn2, 1.0f, z.x, z.y);
  Gen::pair(c2, c3, kMinusTwoLn2, 1.0f, z.z, z.w);
  return z;
}

// ------------------------------------------------------------------------------------------
// K0: initial model.  Every row gets w_(0)[p] = init_std * z(seed; p), momentum 0; lanes beyond P
// (ragged group and row padding) are zeroed in both arenas.  One thread per column group of the
// padded row.
// ------------------------------------------------------------------------------------------
template <typename WT>
__global__ void __launch_bounds__(kThreads)
k_init(WT *__restrict__ w, float *__restrict__ m, int64_t stride, int64_t n_params, int n_devices,
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
// counts, one launch.  Thread = column group; it visits the listed rows one after the other:
// load w and m once, run that device's steps in registers (gradient from the counter-based
// generator), store once.  The next row's loads are issued before the current row's arithmetic.
// The gradient noise grad_std * z is produced directly (the scale is folded into the constants
// of the radius), which differs from rounding z first by about one part in 10^7.
// ------------------------------------------------------------------------------------------
// The first Philox round of a gradient block multiplies the column-group index (fixed per thread)
// and the device id (fixed per row), so it is hoisted: the host folds the device product, the tag
// word and the first round keys into three words per row, the thread keeps the group product, and
// per step the round is two xors.  The host also guarantees that a row's step counter does not
// cross a multiple of 2^32 inside one launch (it splits the call), so the step index is one add.
struct LocalStepArgs {
  int32_t n;
  int32_t row[kMaxDevices];
  int32_t steps[kMaxDevices];
  uint32_t base_lo[kMaxDevices];  // low word of the device's step counter before this call
  uint32_t r1_c0[kMaxDevices];    // hi(M1 * device) ^ key_a[0]      (xor step index -> word 0)
  uint32_t r1_c1[kMaxDevices];    // lo(M1 * device)                                 (word 1)
  uint32_t r1_c2[kMaxDevices];    // (tag | step_hi) ^ key_b[0]   (xor hi(M0 * group) -> word 2)
};

template <typename Gen>
__device__ __forceinline__ void sgd_steps(float4 &w, float4 &m, uint32_t g_hi, uint32_t g_lo,
                                          uint32_t r1_c0, uint32_t r1_c1, uint32_t r1_c2,
                                          uint32_t base_lo, int steps, const PhiloxKeys &keys,
                                          float neg_lr, float mu, float wd, float lg_scale,
                                          float scale2) {
  const uint32_t c2_first = g_hi ^ r1_c2;
  for (int e = 0; e < steps; ++e) {
    uint32_t c0 = r1_c0 ^ (base_lo + (uint32_t)e), c1 = r1_c1, c2 = c2_first, c3 = g_lo;
#pragma unroll
    for (int r = 1; r < 10; ++r) philox_round(c0, c1, c2, c3, keys.a[r], keys.b[r]);
    float4 n;  // grad_std * z
    Gen::pair(c0, c1, lg_scale, scale2, n.x, n.y);
    Gen::pair(c2, c3, lg_scale, scale2, n.z, n.w);
    float g;
    g = fmaf(wd, w.x, n.x); m.x = fmaf(mu, m.x, g); w.x = fmaf(neg_lr, m.x, w.x);
    g = fmaf(wd, w.y, n.y); m.y = fmaf(mu, m.y, g); w.y = fmaf(neg_lr, m.y, w.y);
    g = fmaf(wd, w.z, n.z); m.z = fmaf(mu, m.z, g); w.z = fmaf(neg_lr, m.z, w.z);
    g = fmaf(wd, w.w, n.w); m.w = fmaf(mu, m.w, g); w.w = fmaf(neg_lr, m.w, w.w);
  }
}

template <typename WT, typename Gen>
__global__ void __launch_bounds__(kThreads)
k_local_step(WT *__restrict__ w, float *__restrict__ m, int64_t stride, int64_t n_params,
             LocalStepArgs a, PhiloxKeys keys, float lr, float mu, float wd, float gstd) {
  const int64_t g = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  const int64_t left = n_params - 4 * g;
  if (left <= 0) return;
  const int live = left >= 4 ? 4 : (int)left;
  const unsigned long long gp = (unsigned long long)kPhiloxM0 * (uint32_t)g;
  const uint32_t g_hi = (uint32_t)(gp >> 32), g_lo = (uint32_t)gp;
  const float scale2 = gstd * gstd, lg_scale = kMinusTwoLn2 * scale2, neg_lr = -lr;

  float4 wv = ld_any(w + (int64_t)a.row[0] * stride, g, live);
  float4 mv = ld_any(m + (int64_t)a.row[0] * stride, g, live);
  for (int j = 0; j < a.n; ++j) {
    float4 wn = wv, mn = mv;
    if (j + 1 < a.n) {
      wn = ld_any(w + (int64_t)a.row[j + 1] * stride, g, live);
      mn = ld_any(m + (int64_t)a.row[j + 1] * stride, g, live);
    }
    const int steps = a.steps[j];
    if (steps > 0) {
      sgd_steps<Gen>(wv, mv, g_hi, g_lo, a.r1_c0[j], a.r1_c1[j], a.r1_c2[j], a.base_lo[j], steps,
                     keys, neg_lr, mu, wd, lg_scale, scale2);
      st_any(w + (int64_t)a.row[j] * stride, g, live, wv);
      st_any(m + (int64_t)a.row[j] * stride, g, live, mv);
    }
    wv = wn;
    mv = mn;
  }
}

// ------------------------------------------------------------------------------------------
// K2: fused weighted combination of `nr` rows written to `nw` rows in the same pass.
//   partial aggregation (Eq. 5): read list = write list = the selected devices, weights a_j;
//   global synchronisation (Algorithm 1): read list = {source}, weight 1, write list = receivers.
//   acc = a_0 * w[rd_0];  acc = fma(a_j, w[rd_j], acc) for j = 1 .. nr-1, in list order.
// KR > 0: compile-time read count (all loads of a thread issued before the first multiply);
// KR == 0: any read count, loads issued in batches of 8.  U column groups per thread keep enough
// bytes in flight when the read list is short.
// ------------------------------------------------------------------------------------------
struct CombineArgs {
  int32_t nr;
  int32_t nw;
  int32_t rd[kMaxDevices];
  float a[kMaxDevices];
  int32_t wr[kMaxDevices];
};

template <typename WT, int KR>
__device__ __forceinline__ float4 combine_group(const WT *__restrict__ w, int64_t stride,
                                                const CombineArgs &c, int64_t g, int live) {
  float4 acc;
  if (KR > 0) {
    float4 v[KR > 0 ? KR : 1];
#pragma unroll
    for (int j = 0; j < KR; ++j) v[j] = ld_any(w + (int64_t)c.rd[j] * stride, g, live);
    acc.x = __fmul_rn(c.a[0], v[0].x);
    acc.y = __fmul_rn(c.a[0], v[0].y);
    acc.z = __fmul_rn(c.a[0], v[0].z);
    acc.w = __fmul_rn(c.a[0], v[0].w);
#pragma unroll
    for (int j = 1; j < KR; ++j) {
      acc.x = fmaf(c.a[j], v[j].x, acc.x);
      acc.y = fmaf(c.a[j], v[j].y, acc.y);
      acc.z = fmaf(c.a[j], v[j].z, acc.z);
      acc.w = fmaf(c.a[j], v[j].w, acc.w);
    }
  } else {
    acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int base = 0; base < c.nr; base += 8) {
      float4 v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (base + j < c.nr) v[j] = ld_any(w + (int64_t)c.rd[base + j] * stride, g, live);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if (base + j < c.nr) {
          const float aj = c.a[base + j];
          if (base + j == 0) {
            acc.x = __fmul_rn(aj, v[j].x);
            acc.y = __fmul_rn(aj, v[j].y);
            acc.z = __fmul_rn(aj, v[j].z);
            acc.w = __fmul_rn(aj, v[j].w);
          } else {
            acc.x = fmaf(aj, v[j].x, acc.x);
            acc.y = fmaf(aj, v[j].y, acc.y);
            acc.z = fmaf(aj, v[j].z, acc.z);
            acc.w = fmaf(aj, v[j].w, acc.w);
          }
        }
      }
    }
  }
  return acc;
}

template <typename WT, int KR, int U>
__global__ void __launch_bounds__(kThreads)
k_combine(WT *__restrict__ w, int64_t stride, int64_t n_params, CombineArgs c) {
  const int64_t n_groups = (n_params + 3) >> 2;
  const int64_t g0 = (int64_t)blockIdx.x * (kThreads * U) + threadIdx.x;
  float4 acc[U];
  int live[U];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const int64_t g = g0 + (int64_t)u * kThreads;
    const int64_t left = n_params - 4 * g;
    live[u] = g < n_groups ? (left >= 4 ? 4 : (int)left) : 0;
    if (live[u] > 0) acc[u] = combine_group<WT, KR>(w, stride, c, g, live[u]);
  }
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const int64_t g = g0 + (int64_t)u * kThreads;
    if (live[u] > 0)
      for (int j = 0; j < c.nw; ++j) st_any(w + (int64_t)c.wr[j] * stride, g, live[u], acc[u]);
  }
}

// ------------------------------------------------------------------------------------------
// K3: per-replica squared norm and squared distance to a reference replica.
// Block b works on row b % N and on the column chunks (b / N), (b / N) + lanes, ...; a chunk is
// kThreads * U column groups.  Blocks that are neighbours in launch order work on the same chunk
// of different rows at about the same time, so the reference chunk is fetched from HBM once and
// found in L2 by the others: HBM traffic stays N * P elements.
// Per thread: fp32 sums over the 4*U elements of a chunk in a fixed order, accumulated in fp64
// across chunks; butterfly over the warp and a fixed-order sum over the warps (fp64) give
// partials[which][row][lane].  The block that takes the last ticket sums the partials of each row
// in a fixed order -> out[2N] (norm2 then div2) and resets the ticket.  No block waits for
// another; fixed grid and fixed orders make the result reproducible bit for bit.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
  return v;
}

template <typename WT, int U>
__global__ void __launch_bounds__(kThreads)
k_stats(const WT *__restrict__ w, int64_t stride, int64_t n_params, int n_devices, int ref,
        int lanes, double *__restrict__ partials, unsigned int *__restrict__ ticket,
        float *__restrict__ out) {
  constexpr int kWarps = kThreads / 32;
  __shared__ double s_part[2][kWarps];
  __shared__ bool s_last;
  const int row = blockIdx.x % n_devices;
  const int my_lane = blockIdx.x / n_devices;
  const int64_t n_groups = (n_params + 3) >> 2;
  const int64_t per_chunk = (int64_t)kThreads * U;
  const int64_t n_chunks = (n_groups + per_chunk - 1) / per_chunk;
  const WT *my_row = w + (int64_t)row * stride;
  const WT *ref_row = w + (int64_t)ref * stride;

  double n2 = 0.0, d2 = 0.0;
  for (int64_t chunk = my_lane; chunk < n_chunks; chunk += lanes) {
    const int64_t g0 = chunk * per_chunk + threadIdx.x;
    float4 v[U], r[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int64_t g = g0 + (int64_t)u * kThreads;
      const int64_t left = n_params - 4 * g;
      if (left >= 4) {
        v[u] = ld_group(my_row, g);
        r[u] = ld_group(ref_row, g);
      } else if (left > 0) {
        v[u] = ld_group_ragged(my_row, g, (int)left);
        r[u] = ld_group_ragged(ref_row, g, (int)left);
      } else {
        v[u] = r[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    float a = 0.f, b = 0.f;
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const float dx = v[u].x - r[u].x, dy = v[u].y - r[u].y;
      const float dz = v[u].z - r[u].z, dw = v[u].w - r[u].w;
      a = fmaf(v[u].x, v[u].x, a); a = fmaf(v[u].y, v[u].y, a);
      a = fmaf(v[u].z, v[u].z, a); a = fmaf(v[u].w, v[u].w, a);
      b = fmaf(dx, dx, b); b = fmaf(dy, dy, b);
      b = fmaf(dz, dz, b); b = fmaf(dw, dw, b);
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
    partials[((int64_t)threadIdx.x * n_devices + row) * lanes + my_lane] = s;
    __threadfence();
  }
  __syncthreads();
  if (threadIdx.x == 0) s_last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  for (int t = warp; t < 2 * n_devices; t += kWarps) {  // t = which * N + row
    const double *src = partials + (int64_t)t * lanes;
    double s = 0.0;
    for (int l = lane; l < lanes; l += 32) s += __ldcg(src + l);
    s = warp_sum(s);
    if (lane == 0) out[t] = (float)s;
  }
  if (threadIdx.x == 0) *ticket = 0u;
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
