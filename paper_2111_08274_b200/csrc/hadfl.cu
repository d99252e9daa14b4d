// C ABI of the HADFL round hot path (see include/hadfl.h): handle, argument checks, version
// bookkeeping, kernel launches.  Every step of the path runs in the kernels of kernels.cuh or in
// the host planning arithmetic of selection.cpp; there is no other implementation to fall back to.
#include "../../include/hadfl.h"

#include <cuda_runtime.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <type_traits>
#include <vector>

#include "kernels.cuh"
#include "selection.h"

using namespace hadfl;

struct hadfl_handle {
  hadfl_config cfg;
  int64_t stride = 0;
  void *w = nullptr;
  void *m = nullptr;
  bool own_arena = false;
  cudaStream_t stream = nullptr;
  int device = 0;
  int sm_count = 0;
  PhiloxKeys keys;
  uint32_t version[kMaxDevices];
  uint64_t step_count[kMaxDevices];
  uint8_t avail[kMaxDevices];
  // K3 scratch
  double *d_partials = nullptr;
  unsigned int *d_ticket = nullptr;
  float *d_stats = nullptr;
  int stats_lanes = 0;  // blocks per row of the statistics kernel
  bool stats_valid = false;
  // fused round kernel scratch
  double *d_round_partials = nullptr;        // [round of a batch][2 N][blocks of the launch]
  double *d_round_group_partials = nullptr;  // [round of a batch][2 N][groups of kFinishGroup blocks]
  unsigned int *d_round_ticket = nullptr;    // [round of a batch][1 + groups]: the round's ticket, one per group
  float *d_round_stats = nullptr;            // [round of a batch][2 * kMaxDevices]
  int round_grid = 0;             // blocks of a launch with packs of 8 columns
  int round_grid_half_packs = 0;  // ... with packs of 4 columns (fp32 batches of one step per device)
  bool round_half_packs = false;  // whether such batches take the packs of 4 columns
  int round_batch = kRoundBatchMax;  // most rounds that hadfl_rounds puts into one launch (1: never batch)
  int last_launch_rounds = 0;        // rounds in the most recent launch of the fused round kernel
  int last_launch_pack = 0;          // columns per thread in that launch
  // model backup that overlaps with later rounds: staging row + copy stream
  void *d_backup = nullptr;
  cudaStream_t backup_stream = nullptr;
  cudaEvent_t backup_ready = nullptr, backup_done = nullptr;
  bool backup_in_flight = false;
  float *backup_dst = nullptr;
  int64_t backup_count = 0;
  std::vector<uint16_t> backup_bf16;  // host landing zone when w is stored as bf16
  float sync_beta = 1.0f;  // weight of the received model on global-synchronisation rounds of hadfl_round
  int last_cuda_error = 0;
  uint64_t launches = 0;
};

namespace {

inline size_t elem_size(const hadfl_handle *h) { return h->cfg.dtype == HADFL_DTYPE_BF16 ? 2 : 4; }
inline size_t m_elem_size(const hadfl_handle *h) { return h->cfg.m_dtype == HADFL_DTYPE_BF16 ? 2 : 4; }

// Calls f(parameter storage type, momentum storage type, rounding mode) for the handle's storage
// configuration: fp32 / fp32, or bf16 parameters with fp32 or bf16 momentum, each rounded to
// nearest even (0) or stochastically (1) at the end of a local-update call.
template <typename T>
struct TypeTag {
  using type = T;
};
template <int V>
using IntTag = std::integral_constant<int, V>;

template <typename F>
int for_storage(const hadfl_handle *h, F &&f) {
  if (h->cfg.dtype == HADFL_DTYPE_FP32) return f(TypeTag<float>{}, TypeTag<float>{}, IntTag<0>{});
  const bool stochastic = h->cfg.rounding == HADFL_ROUND_STOCHASTIC;
  if (h->cfg.m_dtype == HADFL_DTYPE_BF16)
    return stochastic ? f(TypeTag<__nv_bfloat16>{}, TypeTag<__nv_bfloat16>{}, IntTag<1>{})
                      : f(TypeTag<__nv_bfloat16>{}, TypeTag<__nv_bfloat16>{}, IntTag<0>{});
  return stochastic ? f(TypeTag<__nv_bfloat16>{}, TypeTag<float>{}, IntTag<1>{})
                    : f(TypeTag<__nv_bfloat16>{}, TypeTag<float>{}, IntTag<0>{});
}

constexpr size_t kBatchSmallArenaBytes = (size_t)64 << 20;  // arenas up to this size are bound by launches, not bytes
constexpr int kRowPerBlockMaxSteps = 2;  // up to this many steps per device a launch is memory-bound: the local update
                                         // then takes one row per block (fp32), the fused round prefetches rows (bf16)
constexpr int kStatsU = 4;  // 16-byte packs per thread and chunk in the statistics kernel
constexpr int64_t kRoundGridCap = 16384;  // most blocks of a fused-round launch (bounds its scratch: 8 MB)

// Columns per thread in the local-update and fused-round kernels: two Philox blocks (two 16-byte
// accesses of fp32 w, one of bf16 w).  Two independent generator chains per thread give the
// scheduler more to issue, and the per-row overhead is spread over twice the elements.
template <typename WT>
struct StepPack {
  static constexpr int E = 8;
};

// Blocks per row ("lanes") of a statistics launch: one wave of resident blocks (8 blocks of 256
// threads per SM) split evenly over the rows, never more blocks per row than there are column
// chunks, and - where the scratch is bounded - never more than max_blocks blocks in all.
int64_t stats_lanes_for(int sm_count, int n_devices, int64_t n_params, int dtype, int64_t max_blocks) {
  const int64_t pack_e = dtype == HADFL_DTYPE_BF16 ? 8 : 4;
  const int64_t packs = (n_params + pack_e - 1) / pack_e;
  const int64_t chunks = (packs + kThreads * kStatsU - 1) / (kThreads * kStatsU);
  int64_t lanes = ((int64_t)sm_count * 8 + n_devices - 1) / n_devices;
  if (lanes > chunks) lanes = chunks;
  if (max_blocks > 0 && lanes * n_devices > max_blocks) lanes = max_blocks / n_devices;
  return lanes < 1 ? 1 : lanes;
}

StepConsts step_consts(const hadfl_handle *h, float lr) {
  StepConsts k;
  k.neg_lr = -lr;
  k.mu = h->cfg.momentum;
  k.wd = h->cfg.weight_decay;
  k.scale2 = h->cfg.grad_std * h->cfg.grad_std;
  k.lg_scale = kMinusTwoLn2 * k.scale2;
  return k;
}

// What the kernels need to know about one device's steps in one launch.
RowStep row_step(const hadfl_handle *h, int dev, uint64_t base, int steps) {
  const uint64_t dp = (uint64_t)kPhiloxM1 * (uint32_t)dev;
  RowStep r;
  r.w_off = (int64_t)dev * h->stride * (int64_t)elem_size(h);
  r.m_off = (int64_t)dev * h->stride * (int64_t)m_elem_size(h);
  r.row = dev;
  r.steps = steps;
  r.base_lo = (uint32_t)base;
  r.r1_c0 = (uint32_t)(dp >> 32) ^ h->keys.a[0];
  r.r1_c1 = (uint32_t)dp;
  r.r1_c2 = (kTagGrad | ((uint32_t)(base >> 32) & 0xFFFFFFu)) ^ h->keys.b[0];
  return r;
}

// ---- debug build: the table of device ranges the kernels may touch --------------------------------
// One table per process (the debug build supports one GPU per process).  The host keeps a mirror,
// publishes it to the device symbol whenever it changes (after the stream has drained, with a
// blocking copy), and reads the error word back in every synchronising call.
#ifdef HADFL_DEBUG
DebugRanges g_debug_host;

int debug_publish() {
  return cudaMemcpyToSymbol(g_debug, &g_debug_host, offsetof(DebugRanges, error)) == cudaSuccess ? 0 : 1;
}
void debug_add(const void *p, size_t nbytes) {
  if (!p || nbytes == 0 || g_debug_host.n >= kDebugRanges) return;
  g_debug_host.lo[g_debug_host.n] = (uint64_t)(uintptr_t)p;
  g_debug_host.hi[g_debug_host.n] = (uint64_t)(uintptr_t)p + nbytes;
  ++g_debug_host.n;
}
void debug_remove(const void *p) {
  for (int r = 0; r < g_debug_host.n; ++r)
    if (g_debug_host.lo[r] == (uint64_t)(uintptr_t)p) {
      --g_debug_host.n;
      g_debug_host.lo[r] = g_debug_host.lo[g_debug_host.n];
      g_debug_host.hi[r] = g_debug_host.hi[g_debug_host.n];
      return;
    }
}
// 0: every access so far was in range; 1: some kernel skipped one (addr = the first such address).
int debug_error(uint64_t *addr) {
  DebugRanges now;
  if (cudaMemcpyFromSymbol(&now, g_debug, sizeof(now)) != cudaSuccess) return 1;
  if (addr) *addr = now.bad_addr;
  return now.error ? 1 : 0;
}
#define HADFL_DEBUG_RESULT()                            \
  do {                                                   \
    if (debug_error(nullptr)) return HADFL_ERR_STATE;    \
  } while (0)
#else
#define HADFL_DEBUG_RESULT() \
  do {                        \
  } while (0)
#endif

#define HADFL_CUDA(h, expr)                       \
  do {                                            \
    cudaError_t e_ = (expr);                      \
    if (e_ != cudaSuccess) {                      \
      (h)->last_cuda_error = (int)e_;             \
      return HADFL_ERR_CUDA;                      \
    }                                             \
  } while (0)

// Makes the handle's device current for the duration of a call.
struct DeviceGuard {
  int prev = -1;
  bool switched = false;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) switched = cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() {
    if (switched) cudaSetDevice(prev);
  }
};

bool distinct_ids(const hadfl_handle *h, const int32_t *ids, int n) {
  if (!ids || n < 1 || n > h->cfg.n_devices) return false;
  uint32_t seen = 0;
  for (int j = 0; j < n; ++j) {
    if (ids[j] < 0 || ids[j] >= h->cfg.n_devices) return false;
    if (seen & (1u << ids[j])) return false;
    seen |= 1u << ids[j];
  }
  return true;
}

void scaled_versions(const hadfl_handle *h, const double *versions, double *x) {
  for (int i = 0; i < h->cfg.n_devices; ++i)
    x[i] = (versions ? versions[i] : (double)h->version[i]) * h->cfg.version_scale;
}

int check_launch(hadfl_handle *h) {
  HADFL_CUDA(h, cudaGetLastError());
  ++h->launches;
  return HADFL_OK;
}

int launch_init(hadfl_handle *h) {
  return for_storage(h, [&](auto wt, auto mt, auto) {
    using WT = typename decltype(wt)::type;
    using MT = typename decltype(mt)::type;
    const int64_t groups = h->stride / 4;
    const unsigned blocks = (unsigned)((groups + kThreads - 1) / kThreads);
    k_init<WT, MT><<<blocks, kThreads, 0, h->stream>>>((WT *)h->w, (MT *)h->m, h->stride,
                                                       h->cfg.n_params, h->cfg.n_devices, h->keys,
                                                       h->cfg.init_std);
    return check_launch(h);
  });
}

int launch_local_step(hadfl_handle *h, const LocalStepArgs &a, float lr) {
  return for_storage(h, [&](auto wt, auto mt, auto rm) {
    using WT = typename decltype(wt)::type;
    using MT = typename decltype(mt)::type;
    constexpr int E = StepPack<WT>::E;
    const int64_t packs = (h->cfg.n_params + E - 1) / E;
    const unsigned blocks = (unsigned)((packs + kThreads - 1) / kThreads);
    // One row per block when the launch is memory-bound throughout (fp32 storage, at most two steps
    // per device); otherwise every block walks over all rows.  Measured at the ResNet-18 size, 8
    // devices: 210 vs 226 us at 1 step, 215 vs 224 us at 2 steps; with 3 or more steps, mixed step
    // counts or bf16 storage the row walk is as fast or faster.
    int max_steps = 0;
    for (int j = 0; j < a.n; ++j) max_steps = a.r[j].steps > max_steps ? a.r[j].steps : max_steps;
    const bool row_per_block = sizeof(WT) == 4 && max_steps <= kRowPerBlockMaxSteps && a.n > 1;
    const dim3 grid(blocks, row_per_block ? (unsigned)a.n : 1u);
    k_local_step<WT, MT, NormalsFast, E, decltype(rm)::value><<<grid, kThreads, 0, h->stream>>>(
        (WT *)h->w, (MT *)h->m, h->cfg.n_params, a, h->keys, step_consts(h, lr));
    return check_launch(h);
  });
}

template <int NR>
int launch_round(hadfl_handle *h, const RoundBatch<NR> &b, float lr) {
  return for_storage(h, [&](auto wt, auto mt, auto rm) {
    using WT = typename decltype(wt)::type;
    using MT = typename decltype(mt)::type;
    const size_t smem = sizeof(float) * kThreads * (size_t)h->cfg.n_devices;
    constexpr int E = StepPack<WT>::E;
    constexpr int RM = decltype(rm)::value;
    const RoundScratch scratch{h->d_round_partials, h->d_round_group_partials, h->d_round_ticket,
                               h->d_round_stats, h->d_stats};
    int max_steps = 0;
    int64_t sum_steps = 0, n_rows = 0;
    for (int r = 0; r < b.n_rounds; ++r)
      for (int j = 0; j < b.round[r].n; ++j) {
        max_steps = b.round[r].r[j].steps > max_steps ? b.round[r].r[j].steps : max_steps;
        sum_steps += b.round[r].r[j].steps;
        ++n_rows;
      }
    bool launched = false;
    if constexpr (sizeof(WT) == 2) {
      // bf16 parameters and at most two steps per device: the build that prefetches the next row
      if (max_steps <= kRowPerBlockMaxSteps) {
        launched = true;
        k_round<WT, MT, NormalsFast, E, RM, true, NR><<<h->round_grid, kThreads, smem, h->stream>>>(
            (WT *)h->w, (MT *)h->m, h->cfg.n_params, b, h->keys, step_consts(h, lr), scratch);
      }
    } else if constexpr (NR > 1) {
      // fp32, a batch of at most 1.5 steps per device on average (and no device beyond two), rows of
      // the resident blocks within the L2: packs of 4 columns (half the rows in flight per block,
      // twice the blocks).  Measured per round, packs of 4 against packs of 8: one step 151 / 181 us
      // (ResNet-18 size, 8 devices) and 447 / 600 us (2^24, 16 devices); steps 1,2,1,2,... 185 / 190,
      // 590 / 625 and 520 / 564 us (VGG-16 size); two steps 217 / 209, 690 / 653, 600 / 590 us.
      if (max_steps <= kRowPerBlockMaxSteps && 2 * sum_steps <= 3 * n_rows && h->round_half_packs) {
        launched = true;
        h->last_launch_pack = E / 2;
        k_round<WT, MT, NormalsFast, E / 2, RM, false, NR><<<h->round_grid_half_packs, kThreads, smem, h->stream>>>(
            (WT *)h->w, (MT *)h->m, h->cfg.n_params, b, h->keys, step_consts(h, lr), scratch);
      }
    }
    if (!launched || sizeof(WT) == 2) h->last_launch_pack = E;
    if (!launched)
      k_round<WT, MT, NormalsFast, E, RM, false, NR><<<h->round_grid, kThreads, smem, h->stream>>>(
          (WT *)h->w, (MT *)h->m, h->cfg.n_params, b, h->keys, step_consts(h, lr), scratch);
    return check_launch(h);
  });
}

template <typename WT, int KR, int U>
int launch_combine_as(hadfl_handle *h, const CombineArgs &c) {
  constexpr int E = Pack16<WT>::E;
  const int64_t per_block = (int64_t)kThreads * U * E;
  const unsigned blocks = (unsigned)((h->cfg.n_params + per_block - 1) / per_block);
  k_combine<WT, KR, U><<<blocks, kThreads, 0, h->stream>>>((WT *)h->w, h->stride,
                                                            h->cfg.n_params, c);
  return check_launch(h);
}

template <typename WT>
int launch_combine(hadfl_handle *h, const CombineArgs &c) {
  switch (c.nr) {
    case 1: return launch_combine_as<WT, 1, 4>(h, c);
    case 2: return launch_combine_as<WT, 2, 4>(h, c);
    case 3: return launch_combine_as<WT, 3, 2>(h, c);
    case 4: return launch_combine_as<WT, 4, 2>(h, c);
    case 8: return launch_combine_as<WT, 8, 1>(h, c);
    case 16: return launch_combine_as<WT, 16, 1>(h, c);
    default: return launch_combine_as<WT, 0, 1>(h, c);
  }
}

template <typename WT>
int launch_stats(hadfl_handle *h, int ref) {
  k_stats<WT, kStatsU><<<h->stats_lanes * h->cfg.n_devices, kThreads, 0, h->stream>>>(
      (const WT *)h->w, h->stride, h->cfg.n_params, h->cfg.n_devices, ref, h->stats_lanes,
      h->d_partials, h->d_ticket, h->d_stats);
  return check_launch(h);
}

int read_row(hadfl_handle *h, int32_t id, float *dst, int64_t count, bool momentum) {
  if (!h) return HADFL_ERR_INVALID;
  if (!dst || id < 0 || id >= h->cfg.n_devices || count < 0 || count > h->cfg.n_params)
    return HADFL_ERR_INVALID;
  DeviceGuard guard(h->device);
  if (count == 0) {
    HADFL_CUDA(h, cudaStreamSynchronize(h->stream));
    HADFL_DEBUG_RESULT();
    return HADFL_OK;
  }
  const void *arena = momentum ? h->m : h->w;
  if ((momentum ? m_elem_size(h) : elem_size(h)) == 4) {
    const float *src = (const float *)arena + (int64_t)id * h->stride;
    HADFL_CUDA(h, cudaMemcpyAsync(dst, src, sizeof(float) * (size_t)count, cudaMemcpyDeviceToHost,
                                  h->stream));
    HADFL_CUDA(h, cudaStreamSynchronize(h->stream));
    HADFL_DEBUG_RESULT();
    return HADFL_OK;
  }
  std::vector<uint16_t> tmp((size_t)count);
  const uint16_t *src = (const uint16_t *)arena + (int64_t)id * h->stride;
  HADFL_CUDA(h, cudaMemcpyAsync(tmp.data(), src, 2 * (size_t)count, cudaMemcpyDeviceToHost, h->stream));
  HADFL_CUDA(h, cudaStreamSynchronize(h->stream));
  HADFL_DEBUG_RESULT();
  for (int64_t p = 0; p < count; ++p) {
    const uint32_t bits = (uint32_t)tmp[(size_t)p] << 16;
    memcpy(dst + p, &bits, 4);
  }
  return HADFL_OK;
}

uint16_t bf16_bits_rn(float v) {
  uint32_t bits;
  memcpy(&bits, &v, 4);
  if ((bits & 0x7F800000u) == 0x7F800000u) return (uint16_t)((bits >> 16) | ((bits & 0x007FFFFFu) ? 0x40u : 0u));
  return (uint16_t)((bits + 0x7FFFu + ((bits >> 16) & 1u)) >> 16);
}

int write_row(hadfl_handle *h, int32_t id, const float *src, int64_t count, bool momentum) {
  if (!h) return HADFL_ERR_INVALID;
  if (!src || id < 0 || id >= h->cfg.n_devices || count < 0 || count > h->cfg.n_params)
    return HADFL_ERR_INVALID;
  if (count == 0) return HADFL_OK;
  DeviceGuard guard(h->device);
  // The copy is ordered on the stream; waiting for it lets the caller reuse src at once.
  void *arena = momentum ? h->m : h->w;
  if ((momentum ? m_elem_size(h) : elem_size(h)) == 4) {
    float *dst = (float *)arena + (int64_t)id * h->stride;
    HADFL_CUDA(h, cudaMemcpyAsync(dst, src, sizeof(float) * (size_t)count, cudaMemcpyHostToDevice,
                                  h->stream));
    HADFL_CUDA(h, cudaStreamSynchronize(h->stream));
    return HADFL_OK;
  }
  std::vector<uint16_t> tmp((size_t)count);
  for (int64_t p = 0; p < count; ++p) tmp[(size_t)p] = bf16_bits_rn(src[p]);
  uint16_t *dst = (uint16_t *)arena + (int64_t)id * h->stride;
  HADFL_CUDA(h, cudaMemcpyAsync(dst, tmp.data(), 2 * (size_t)count, cudaMemcpyHostToDevice, h->stream));
  HADFL_CUDA(h, cudaStreamSynchronize(h->stream));
  return HADFL_OK;
}

}  // namespace

extern "C" {

int hadfl_init(const hadfl_config *cfg, hadfl_handle **out) {
  if (!cfg || !out) return HADFL_ERR_INVALID;
  *out = nullptr;
  if (cfg->n_devices < 1 || cfg->n_devices > HADFL_MAX_DEVICES) return HADFL_ERR_INVALID;
  if (cfg->n_params < 1 || cfg->n_params > ((int64_t)1 << 34) - 4) return HADFL_ERR_INVALID;
  if (cfg->dtype != HADFL_DTYPE_FP32 && cfg->dtype != HADFL_DTYPE_BF16) return HADFL_ERR_INVALID;
  if (cfg->m_dtype != HADFL_DTYPE_FP32 && cfg->m_dtype != HADFL_DTYPE_BF16) return HADFL_ERR_INVALID;
  if (cfg->rounding != HADFL_ROUND_NEAREST && cfg->rounding != HADFL_ROUND_STOCHASTIC)
    return HADFL_ERR_INVALID;
  // bf16 momentum and stochastic rounding are options of bf16 parameter storage
  if (cfg->dtype == HADFL_DTYPE_FP32 && (cfg->m_dtype != HADFL_DTYPE_FP32 || cfg->rounding != HADFL_ROUND_NEAREST))
    return HADFL_ERR_INVALID;
  if (cfg->weight_mode != HADFL_WEIGHTS_UNIFORM && cfg->weight_mode != HADFL_WEIGHTS_VERSION)
    return HADFL_ERR_INVALID;
  if ((cfg->w_ptr == nullptr) != (cfg->m_ptr == nullptr)) return HADFL_ERR_INVALID;
  if (!(cfg->version_scale > 0.0)) return HADFL_ERR_INVALID;
  if (!(cfg->grad_std >= 0.0f)) return HADFL_ERR_INVALID;
  int64_t stride = cfg->row_stride_elems;
  if (stride == 0) stride = (cfg->n_params + 31) / 32 * 32;
  if (stride < cfg->n_params || stride % 8 != 0) return HADFL_ERR_INVALID;
  if (cfg->w_ptr && (((uintptr_t)cfg->w_ptr | (uintptr_t)cfg->m_ptr) & 15u)) return HADFL_ERR_INVALID;

  hadfl_handle *h = new (std::nothrow) hadfl_handle;
  if (!h) return HADFL_ERR_STATE;
  h->cfg = *cfg;
  h->stride = stride;
  h->stream = (cudaStream_t)cfg->cuda_stream;
  h->keys = expand_keys(cfg->seed);
  for (int i = 0; i < kMaxDevices; ++i) {
    h->version[i] = 0;
    h->step_count[i] = 0;
    h->avail[i] = 1;
  }
  // From here on failures are CUDA failures; the handle is returned so that the caller can read
  // the error code, and must still be destroyed.
  *out = h;
  HADFL_CUDA(h, cudaGetDevice(&h->device));
  HADFL_CUDA(h, cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device));
  const size_t elems = (size_t)cfg->n_devices * (size_t)stride;
  if (!cfg->w_ptr) {
    h->own_arena = true;
    HADFL_CUDA(h, cudaMalloc(&h->w, elems * elem_size(h)));
    HADFL_CUDA(h, cudaMalloc(&h->m, elems * m_elem_size(h)));
  } else {
    h->w = cfg->w_ptr;
    h->m = cfg->m_ptr;
  }
  const int64_t lanes = stats_lanes_for(h->sm_count, cfg->n_devices, cfg->n_params, cfg->dtype, 0);
  h->stats_lanes = (int)lanes;
  HADFL_CUDA(h, cudaMalloc((void **)&h->d_partials,
                           sizeof(double) * 2 * (size_t)cfg->n_devices * (size_t)lanes));
  HADFL_CUDA(h, cudaMalloc((void **)&h->d_ticket, sizeof(unsigned int)));
  HADFL_CUDA(h, cudaMalloc((void **)&h->d_stats, sizeof(float) * 2 * kMaxDevices));
  // Fused round kernel: one block per chunk of kThreads packs (8 columns each) up to kRoundGridCap
  // blocks, beyond which the blocks stride over the chunks.  Measured on the workloads' sizes, a grid
  // of many short blocks beats one resident wave by 7-15 % with several steps per device and is
  // equal at one step (caps of 592 / 1184 / 2368 / 4736 / 16384 blocks at the ResNet-18 size, 8
  // devices, uniform 1..8 steps: 401 / 378 / 371 / 371 / 373 us).
  {
    const int64_t round_packs = (cfg->n_params + 7) / 8;
    const int64_t need = (round_packs + kThreads - 1) / kThreads;
    h->round_grid = (int)(need < kRoundGridCap ? need : kRoundGridCap);
    const int64_t need_half = ((cfg->n_params + 3) / 4 + kThreads - 1) / kThreads;
    h->round_grid_half_packs = (int)(need_half < kRoundGridCap ? need_half : kRoundGridCap);
    // Batches of rounds with fp32 storage and one step per device take packs of 4 columns while the
    // rows that the resident blocks hold at one time (4 blocks per SM x N devices x 1024 columns x
    // 8 bytes) stay within 80 % of the L2 and the arena is not a small one (measured at one step per
    // device, 8 rounds per launch: 151 against 181 us per round with 8 devices at the ResNet-18 size,
    // 447 against 600 us with 16 devices and 2^24 parameters; with 32 devices - 155 MB of rows -
    // 2065 against 1943 us, and 19.1 against 17.5 us at 2^18 parameters, where launches are the cost).
    int l2_bytes = 0;
    HADFL_CUDA(h, cudaDeviceGetAttribute(&l2_bytes, cudaDevAttrL2CacheSize, h->device));
    const double resident_rows = 4.0 * h->sm_count * cfg->n_devices * (kThreads * 4.0) * 8.0;
    h->round_half_packs = cfg->dtype == HADFL_DTYPE_FP32 && resident_rows <= 0.8 * l2_bytes &&
                          (size_t)cfg->n_devices * (size_t)cfg->n_params * 8 > kBatchSmallArenaBytes;
  }
  const int scratch_grid = h->round_grid_half_packs > h->round_grid ? h->round_grid_half_packs : h->round_grid;
  const size_t n_groups = (size_t)((scratch_grid + kFinishGroup - 1) / kFinishGroup);
  const size_t round_vals = (size_t)kRoundBatchMax * 2 * (size_t)cfg->n_devices;
  HADFL_CUDA(h, cudaMalloc((void **)&h->d_round_partials, sizeof(double) * round_vals * (size_t)scratch_grid));
  HADFL_CUDA(h, cudaMalloc((void **)&h->d_round_group_partials, sizeof(double) * round_vals * n_groups));
  HADFL_CUDA(h, cudaMalloc((void **)&h->d_round_ticket, sizeof(unsigned int) * kRoundBatchMax * (1 + n_groups)));
  HADFL_CUDA(h, cudaMalloc((void **)&h->d_round_stats, sizeof(float) * kRoundBatchMax * 2 * kMaxDevices));
  HADFL_CUDA(h, cudaMemsetAsync(h->d_round_ticket, 0, sizeof(unsigned int) * kRoundBatchMax * (1 + n_groups),
                                h->stream));
  HADFL_CUDA(h, cudaMemsetAsync(h->d_round_stats, 0, sizeof(float) * kRoundBatchMax * 2 * kMaxDevices, h->stream));
  HADFL_CUDA(h, cudaMemsetAsync(h->d_ticket, 0, sizeof(unsigned int), h->stream));
  HADFL_CUDA(h, cudaMemsetAsync(h->d_stats, 0, sizeof(float) * 2 * kMaxDevices, h->stream));
#ifdef HADFL_DEBUG
  debug_add(h->w, elems * elem_size(h));
  debug_add(h->m, elems * m_elem_size(h));
  debug_add(h->d_partials, sizeof(double) * 2 * (size_t)cfg->n_devices * (size_t)lanes);
  debug_add(h->d_stats, sizeof(float) * 2 * kMaxDevices);
  debug_add(h->d_round_partials, sizeof(double) * round_vals * (size_t)scratch_grid);
  debug_add(h->d_round_group_partials, sizeof(double) * round_vals * n_groups);
  debug_add(h->d_round_stats, sizeof(float) * kRoundBatchMax * 2 * kMaxDevices);
  HADFL_CUDA(h, cudaDeviceSynchronize());
  if (debug_publish()) return HADFL_ERR_CUDA;
#endif
  return launch_init(h);
}

int hadfl_destroy(hadfl_handle *h) {
  if (!h) return HADFL_OK;
  DeviceGuard guard(h->device);
  hadfl_backup_wait(h);
  cudaStreamSynchronize(h->stream);
#ifdef HADFL_DEBUG
  cudaDeviceSynchronize();
  debug_remove(h->w);
  debug_remove(h->m);
  debug_remove(h->d_partials);
  debug_remove(h->d_stats);
  debug_remove(h->d_round_partials);
  debug_remove(h->d_round_group_partials);
  debug_remove(h->d_round_stats);
  debug_publish();
#endif
  if (h->own_arena) {
    cudaFree(h->w);
    cudaFree(h->m);
  }
  cudaFree(h->d_partials);
  cudaFree(h->d_ticket);
  cudaFree(h->d_stats);
  cudaFree(h->d_round_partials);
  cudaFree(h->d_round_group_partials);
  cudaFree(h->d_round_ticket);
  cudaFree(h->d_round_stats);
  if (h->backup_stream) cudaStreamSynchronize(h->backup_stream);
  cudaFree(h->d_backup);
  if (h->backup_ready) cudaEventDestroy(h->backup_ready);
  if (h->backup_done) cudaEventDestroy(h->backup_done);
  if (h->backup_stream) cudaStreamDestroy(h->backup_stream);
  delete h;
  return HADFL_OK;
}

int hadfl_local_step(hadfl_handle *h, const int32_t *device_ids, const int32_t *steps, int32_t n,
                     float lr) {
  if (!h) return HADFL_ERR_INVALID;
  if (!steps || !distinct_ids(h, device_ids, n)) return HADFL_ERR_INVALID;
  for (int j = 0; j < n; ++j)
    if (steps[j] < 0) return HADFL_ERR_INVALID;
  for (int j = 0; j < n; ++j)
    if ((h->step_count[device_ids[j]] + (uint64_t)steps[j]) >> 56)
      return HADFL_ERR_STATE;  // a device's gradient stream has 2^56 steps
  DeviceGuard guard(h->device);
  // One launch covers every listed device.  A second one is needed only when some device's step
  // counter crosses a multiple of 2^32 inside this call (once in 4 billion steps): the kernel
  // takes the high word of the step index as fixed per launch.
  int done[kMaxDevices];
  for (int j = 0; j < n; ++j) done[j] = 0;
  for (;;) {
    LocalStepArgs a;
    memset(&a, 0, sizeof(a));
    bool more = false;
    for (int j = 0; j < n; ++j) {
      const int dev = device_ids[j];
      const uint64_t base = h->step_count[dev] + (uint64_t)done[j];
      const uint64_t room = ((uint64_t)1 << 32) - (base & 0xFFFFFFFFull);
      int take = steps[j] - done[j];
      if ((uint64_t)take > room) {
        take = (int)room;
        more = true;
      }
      if (take == 0) continue;  // nothing to run (a device listed with 0 steps is not touched)
      a.r[a.n++] = row_step(h, dev, base, take);
      done[j] += take;
    }
    if (a.n > 0) {
      const int rc = launch_local_step(h, a, lr);
      if (rc != HADFL_OK) return rc;
    }
    if (!more) break;
  }
  for (int j = 0; j < n; ++j) {
    h->step_count[device_ids[j]] += (uint64_t)steps[j];
    h->version[device_ids[j]] += (uint32_t)steps[j];
  }
  return HADFL_OK;
}

int hadfl_select(hadfl_handle *h, int64_t round, const double *versions, uint64_t seed, int32_t k,
                 int32_t *out_selected) {
  if (!h || !out_selected) return HADFL_ERR_INVALID;
  double x[kMaxDevices];
  scaled_versions(h, versions, x);
  return selection_draw(x, h->avail, h->cfg.n_devices, round, seed, k, out_selected)
             ? HADFL_OK
             : HADFL_ERR_INVALID;
}

int hadfl_select_probs(hadfl_handle *h, const double *versions, double *out_P) {
  if (!h || !out_P) return HADFL_ERR_INVALID;
  double x[kMaxDevices];
  scaled_versions(h, versions, x);
  return selection_probs(x, h->avail, h->cfg.n_devices, out_P) ? HADFL_OK : HADFL_ERR_INVALID;
}

int hadfl_select_probs_after(hadfl_handle *h, const int32_t *device_ids, const int32_t *steps, int32_t n,
                             double *out_P) {
  if (!h || !out_P || !steps || !distinct_ids(h, device_ids, n)) return HADFL_ERR_INVALID;
  double x[kMaxDevices];
  for (int i = 0; i < h->cfg.n_devices; ++i) x[i] = (double)h->version[i];
  for (int j = 0; j < n; ++j) {
    if (steps[j] < 0) return HADFL_ERR_INVALID;
    x[device_ids[j]] = (double)(h->version[device_ids[j]] + (uint32_t)steps[j]);
  }
  for (int i = 0; i < h->cfg.n_devices; ++i) x[i] *= h->cfg.version_scale;
  return selection_probs(x, h->avail, h->cfg.n_devices, out_P) ? HADFL_OK : HADFL_ERR_INVALID;
}

int hadfl_aggregation_weights(hadfl_handle *h, const int32_t *selected, int32_t k,
                              const double *versions, float *out_a) {
  if (!h || !out_a || !distinct_ids(h, selected, k)) return HADFL_ERR_INVALID;
  double x[kMaxDevices];
  scaled_versions(h, versions, x);
  aggregation_weights(h->cfg.weight_mode, x, h->avail, h->cfg.n_devices, selected, k, out_a);
  return HADFL_OK;
}

int hadfl_aggregate(hadfl_handle *h, const int32_t *selected, int32_t k, const double *versions) {
  if (!h || !distinct_ids(h, selected, k)) return HADFL_ERR_INVALID;
  CombineArgs c;
  memset(&c, 0, sizeof(c));
  c.nr = c.nw = k;
  double x[kMaxDevices];
  scaled_versions(h, versions, x);
  aggregation_weights(h->cfg.weight_mode, x, h->avail, h->cfg.n_devices, selected, k, c.a);
  for (int j = 0; j < k; ++j) c.rd[j] = c.wr[j] = selected[j];
  if (k > 1) {  // a single selected device is a no-op (a_0 = 1): nothing to launch
    DeviceGuard guard(h->device);
    const int rc = h->cfg.dtype == HADFL_DTYPE_BF16 ? launch_combine<__nv_bfloat16>(h, c)
                                                    : launch_combine<float>(h, c);
    if (rc != HADFL_OK) return rc;
  }
  uint32_t vmax = 0;
  for (int j = 0; j < k; ++j) vmax = h->version[selected[j]] > vmax ? h->version[selected[j]] : vmax;
  for (int j = 0; j < k; ++j) h->version[selected[j]] = vmax;
  return HADFL_OK;
}

int hadfl_broadcast(hadfl_handle *h, int32_t src, const int32_t *dst_ids, int32_t n) {
  if (!h || src < 0 || src >= h->cfg.n_devices || n < 0) return HADFL_ERR_INVALID;
  if (n == 0) return HADFL_OK;
  if (!distinct_ids(h, dst_ids, n)) return HADFL_ERR_INVALID;
  for (int j = 0; j < n; ++j)
    if (dst_ids[j] == src) return HADFL_ERR_INVALID;
  CombineArgs c;
  memset(&c, 0, sizeof(c));
  c.nr = 1;
  c.nw = n;
  c.rd[0] = src;
  c.a[0] = 1.0f;
  for (int j = 0; j < n; ++j) c.wr[j] = dst_ids[j];
  DeviceGuard guard(h->device);
  const int rc = h->cfg.dtype == HADFL_DTYPE_BF16 ? launch_combine<__nv_bfloat16>(h, c)
                                                  : launch_combine<float>(h, c);
  if (rc != HADFL_OK) return rc;
  for (int j = 0; j < n; ++j) h->version[dst_ids[j]] = h->version[src];
  return HADFL_OK;
}

int hadfl_integrate(hadfl_handle *h, int32_t src, const int32_t *dst_ids, int32_t n, float beta) {
  if (!h || src < 0 || src >= h->cfg.n_devices || n < 0) return HADFL_ERR_INVALID;
  if (!(beta >= 0.0f && beta <= 1.0f)) return HADFL_ERR_INVALID;
  if (n == 0) return HADFL_OK;
  if (!distinct_ids(h, dst_ids, n)) return HADFL_ERR_INVALID;
  for (int j = 0; j < n; ++j)
    if (dst_ids[j] == src) return HADFL_ERR_INVALID;
  MixArgs a;
  memset(&a, 0, sizeof(a));
  a.n = n;
  a.src = src;
  a.beta = beta;
  a.one_minus_beta = 1.0f - beta;
  for (int j = 0; j < n; ++j) a.dst[j] = dst_ids[j];
  {
    DeviceGuard guard(h->device);
    constexpr int U = 2;
    const int64_t pack_e = h->cfg.dtype == HADFL_DTYPE_BF16 ? 8 : 4;
    const int64_t per_block = (int64_t)kThreads * U * pack_e;
    const unsigned blocks = (unsigned)((h->cfg.n_params + per_block - 1) / per_block);
    if (h->cfg.dtype == HADFL_DTYPE_BF16)
      k_integrate<__nv_bfloat16, U><<<blocks, kThreads, 0, h->stream>>>((__nv_bfloat16 *)h->w, h->stride,
                                                                     h->cfg.n_params, a);
    else
      k_integrate<float, U><<<blocks, kThreads, 0, h->stream>>>((float *)h->w, h->stride,
                                                             h->cfg.n_params, a);
    const int rc = check_launch(h);
    if (rc != HADFL_OK) return rc;
  }
  for (int j = 0; j < n; ++j) {
    uint32_t &v = h->version[dst_ids[j]];
    if (beta == 1.0f || h->version[src] > v) v = h->version[src];
  }
  return HADFL_OK;
}

int hadfl_set_sync_beta(hadfl_handle *h, float beta) {
  if (!h || !(beta >= 0.0f && beta <= 1.0f)) return HADFL_ERR_INVALID;
  h->sync_beta = beta;
  return HADFL_OK;
}

namespace {

// One round as the host plans it before anything is enqueued: the steps per row, the selection
// (which sees the versions as they will be after the local steps) and the kernel's arguments.
struct RoundPlan {
  int row_steps[kMaxDevices];
  int32_t sel[kMaxDevices];
  bool crosses;  // a step counter crosses a multiple of 2^32 in this round
  RoundArgs a;
};

int plan_round(hadfl_handle *h, const int32_t *device_ids, const int32_t *steps, int32_t n, int64_t round,
               const double *versions, uint64_t seed, int32_t k, int32_t sync_all, RoundPlan &pl) {
  if (!steps || !distinct_ids(h, device_ids, n)) return HADFL_ERR_INVALID;
  const int N = h->cfg.n_devices;
  for (int i = 0; i < N; ++i) pl.row_steps[i] = 0;
  pl.crosses = false;
  for (int j = 0; j < n; ++j) {
    if (steps[j] < 0) return HADFL_ERR_INVALID;
    const uint64_t base = h->step_count[device_ids[j]];
    if ((base + (uint64_t)steps[j]) >> 56) return HADFL_ERR_STATE;
    if ((base & 0xFFFFFFFFull) + (uint64_t)steps[j] > ((uint64_t)1 << 32)) pl.crosses = true;
    pl.row_steps[device_ids[j]] = steps[j];
  }
  double x[kMaxDevices];
  for (int i = 0; i < N; ++i)
    x[i] = (versions ? versions[i] : (double)(h->version[i] + (uint32_t)pl.row_steps[i])) *
           h->cfg.version_scale;
  if (!selection_draw(x, h->avail, N, round, seed, k, pl.sel)) return HADFL_ERR_INVALID;
  if (pl.crosses) return HADFL_OK;

  RoundArgs &a = pl.a;
  memset(&a, 0, sizeof(a));
  a.n = N;
  a.k = k;
  a.write_all = sync_all ? (h->sync_beta == 1.0f ? 1 : 2) : 0;
  a.beta = h->sync_beta;
  a.one_minus_beta = 1.0f - h->sync_beta;
  aggregation_weights(h->cfg.weight_mode, x, h->avail, N, pl.sel, k, a.a);
  uint32_t in_sel = 0;
  int pos = 0;
  for (int j = 0; j < k; ++j) {
    a.r[pos++] = row_step(h, pl.sel[j], h->step_count[pl.sel[j]], pl.row_steps[pl.sel[j]]);
    in_sel |= 1u << pl.sel[j];
  }
  for (int i = 0; i < N; ++i)
    if (!(in_sel & (1u << i))) a.r[pos++] = row_step(h, i, h->step_count[i], pl.row_steps[i]);
  return HADFL_OK;
}

// The host's mirror of the counters after a planned round (fused path).
void commit_round(hadfl_handle *h, const RoundPlan &pl, int32_t k, int32_t sync_all) {
  const int N = h->cfg.n_devices;
  for (int i = 0; i < N; ++i) {
    h->step_count[i] += (uint64_t)pl.row_steps[i];
    h->version[i] += (uint32_t)pl.row_steps[i];
  }
  uint32_t vmax = 0;
  for (int j = 0; j < k; ++j) vmax = h->version[pl.sel[j]] > vmax ? h->version[pl.sel[j]] : vmax;
  for (int j = 0; j < k; ++j) h->version[pl.sel[j]] = vmax;
  if (sync_all)
    for (int i = 0; i < N; ++i)
      if (h->sync_beta == 1.0f || vmax > h->version[i]) h->version[i] = vmax;
}

// A round whose step counters cross a multiple of 2^32 (once in 4 billion steps): the separate
// kernels, which split the launch.
int round_by_separate_calls(hadfl_handle *h, const int32_t *device_ids, const int32_t *steps, int32_t n,
                            float lr, const double *versions, int32_t k, int32_t sync_all,
                            const int32_t *sel) {
  const int N = h->cfg.n_devices;
  int rc = hadfl_local_step(h, device_ids, steps, n, lr);
  if (rc == HADFL_OK) rc = hadfl_aggregate(h, sel, k, versions);
  if (rc == HADFL_OK && sync_all) {
    int32_t others[kMaxDevices];
    int n_others = 0;
    uint32_t in_sel = 0;
    for (int j = 0; j < k; ++j) in_sel |= 1u << sel[j];
    for (int i = 0; i < N; ++i)
      if (!(in_sel & (1u << i))) others[n_others++] = i;
    rc = h->sync_beta == 1.0f ? hadfl_broadcast(h, sel[0], others, n_others)
                              : hadfl_integrate(h, sel[0], others, n_others, h->sync_beta);
  }
  if (rc == HADFL_OK) rc = hadfl_stats_enqueue(h, sel[0]);
  if (rc == HADFL_OK) h->last_launch_rounds = 0;
  return rc;
}

// Whether hadfl_rounds may put a planned round into a launch together with its neighbours.  A
// batch pays where a round is bound by memory or by the launch itself: every device runs at most
// kRowPerBlockMaxSteps steps, or the arena is small against the L2.  With more steps per device
// the rounds are bound by arithmetic and the batch's indexed arguments cost what L2 saves
// (measured: 0 ... -3 %), so those rounds are launched one by one; the same holds for stochastic
// rounding, which draws a second random block per pack and call (measured: -3 ... -5 %).
bool batchable(const hadfl_handle *h, const RoundPlan &pl) {
  if (h->round_batch <= 1) return false;
  const size_t arena = (size_t)h->cfg.n_devices * (size_t)h->cfg.n_params * (elem_size(h) + m_elem_size(h));
  if (arena <= kBatchSmallArenaBytes) return true;
  if (h->cfg.rounding == HADFL_ROUND_STOCHASTIC) return false;
  for (int i = 0; i < h->cfg.n_devices; ++i)
    if (pl.row_steps[i] > kRowPerBlockMaxSteps) return false;
  return true;
}

}  // namespace

int hadfl_round(hadfl_handle *h, const int32_t *device_ids, const int32_t *steps, int32_t n, float lr,
                int64_t round, const double *versions, uint64_t seed, int32_t k, int32_t sync_all,
                int32_t *out_selected) {
  if (!h || !out_selected) return HADFL_ERR_INVALID;
  RoundPlan pl;
  int rc = plan_round(h, device_ids, steps, n, round, versions, seed, k, sync_all, pl);
  if (rc != HADFL_OK) return rc;
  if (pl.crosses) {
    rc = round_by_separate_calls(h, device_ids, steps, n, lr, versions, k, sync_all, pl.sel);
    if (rc != HADFL_OK) return rc;
  } else {
    RoundBatch<1> b;
    b.n_rounds = 1;
    b.round[0] = pl.a;
    {
      DeviceGuard guard(h->device);
      rc = launch_round(h, b, lr);
      if (rc != HADFL_OK) return rc;
    }
    commit_round(h, pl, k, sync_all);
    h->stats_valid = true;
    h->last_launch_rounds = 1;
  }
  for (int j = 0; j < k; ++j) out_selected[j] = pl.sel[j];
  return HADFL_OK;
}

int hadfl_rounds(hadfl_handle *h, int64_t first_round, int32_t n_rounds, const int32_t *steps, float lr,
                 uint64_t seed, int32_t k, int32_t sync_every, int32_t *out_selected) {
  if (!h || !steps || n_rounds < 0 || sync_every < 0) return HADFL_ERR_INVALID;
  const int N = h->cfg.n_devices;
  int32_t ids[kMaxDevices];
  for (int i = 0; i < N; ++i) ids[i] = i;
  // Rounds are planned on the host one after the other (each sees the counters the previous one
  // leaves).  Rounds that gain from it are collected into batches of up to round_batch rounds per
  // launch; the others are launched one by one.
  RoundBatch<kRoundBatchMax> batch;
  batch.n_rounds = 0;
  uint32_t version_before[kMaxDevices];  // the counters before the pending batch, should its launch fail
  uint64_t step_count_before[kMaxDevices];
  auto flush = [&]() -> int {
    if (batch.n_rounds == 0) return HADFL_OK;
    int rc;
    {
      DeviceGuard guard(h->device);
      if (batch.n_rounds == 1) {
        RoundBatch<1> one;
        one.n_rounds = 1;
        one.round[0] = batch.round[0];
        rc = launch_round(h, one, lr);
      } else {
        rc = launch_round(h, batch, lr);
      }
    }
    if (rc == HADFL_OK) {
      h->stats_valid = true;
      h->last_launch_rounds = batch.n_rounds;
    } else {
      memcpy(h->version, version_before, sizeof(version_before));
      memcpy(h->step_count, step_count_before, sizeof(step_count_before));
    }
    batch.n_rounds = 0;
    return rc;
  };
  for (int32_t i = 0; i < n_rounds; ++i) {
    const int64_t r = first_round + i;
    const int32_t sync = sync_every > 0 && (r + 1) % sync_every == 0;
    const int32_t *round_steps = steps + (int64_t)i * N;
    RoundPlan pl;
    int rc = plan_round(h, ids, round_steps, N, r, nullptr, seed, k, sync, pl);
    if (rc != HADFL_OK) {
      const int rc_flush = flush();  // what was planned before the bad round still runs
      return rc_flush != HADFL_OK ? rc_flush : rc;
    }
    if (pl.crosses) {
      rc = flush();
      if (rc == HADFL_OK) rc = round_by_separate_calls(h, ids, round_steps, N, lr, nullptr, k, sync, pl.sel);
    } else {
      if (!batchable(h, pl)) rc = flush();
      if (rc == HADFL_OK) {
        if (batch.n_rounds == 0) {
          memcpy(version_before, h->version, sizeof(version_before));
          memcpy(step_count_before, h->step_count, sizeof(step_count_before));
        }
        batch.round[batch.n_rounds++] = pl.a;
        commit_round(h, pl, k, sync);
        if (!batchable(h, pl) || batch.n_rounds >= h->round_batch) rc = flush();
      }
    }
    if (rc != HADFL_OK) return rc;
    if (out_selected)
      for (int j = 0; j < k; ++j) out_selected[(int64_t)i * k + j] = pl.sel[j];
  }
  return flush();
}

int hadfl_set_round_batch(hadfl_handle *h, int32_t max_rounds) {
  if (!h || max_rounds < 1 || max_rounds > kRoundBatchMax) return HADFL_ERR_INVALID;
  h->round_batch = max_rounds;
  return HADFL_OK;
}

int32_t hadfl_round_batch(const hadfl_handle *h) { return h ? h->round_batch : 0; }
int32_t hadfl_last_round_pack(const hadfl_handle *h) { return h ? h->last_launch_pack : 0; }

int hadfl_stats_read_round(hadfl_handle *h, int32_t back, float *out_norm2, float *out_div2) {
  if (!h || !out_norm2 || !out_div2 || back < 0) return HADFL_ERR_INVALID;
  if (back == 0) return hadfl_stats_read(h, out_norm2, out_div2);
  if (!h->stats_valid || back >= h->last_launch_rounds) return HADFL_ERR_STATE;
  DeviceGuard guard(h->device);
  float buf[2 * kMaxDevices];
  const int n = h->cfg.n_devices;
  const float *src = h->d_round_stats + (size_t)(h->last_launch_rounds - 1 - back) * 2 * kMaxDevices;
  HADFL_CUDA(h, cudaMemcpyAsync(buf, src, sizeof(float) * 2 * (size_t)n, cudaMemcpyDeviceToHost, h->stream));
  HADFL_CUDA(h, cudaStreamSynchronize(h->stream));
  HADFL_DEBUG_RESULT();
  memcpy(out_norm2, buf, sizeof(float) * (size_t)n);
  memcpy(out_div2, buf + n, sizeof(float) * (size_t)n);
  return HADFL_OK;
}

int hadfl_stats_enqueue(hadfl_handle *h, int32_t ref_device) {
  if (!h || ref_device < 0 || ref_device >= h->cfg.n_devices) return HADFL_ERR_INVALID;
  DeviceGuard guard(h->device);
  const int rc = h->cfg.dtype == HADFL_DTYPE_BF16 ? launch_stats<__nv_bfloat16>(h, ref_device)
                                                  : launch_stats<float>(h, ref_device);
  if (rc == HADFL_OK) h->stats_valid = true;
  return rc;
}

int hadfl_stats_read(hadfl_handle *h, float *out_norm2, float *out_div2) {
  if (!h || !out_norm2 || !out_div2) return HADFL_ERR_INVALID;
  if (!h->stats_valid) return HADFL_ERR_STATE;
  DeviceGuard guard(h->device);
  float buf[2 * kMaxDevices];
  const int n = h->cfg.n_devices;
  HADFL_CUDA(h, cudaMemcpyAsync(buf, h->d_stats, sizeof(float) * 2 * (size_t)n,
                                cudaMemcpyDeviceToHost, h->stream));
  HADFL_CUDA(h, cudaStreamSynchronize(h->stream));
  HADFL_DEBUG_RESULT();
  memcpy(out_norm2, buf, sizeof(float) * (size_t)n);
  memcpy(out_div2, buf + n, sizeof(float) * (size_t)n);
  return HADFL_OK;
}

int hadfl_stats(hadfl_handle *h, int32_t ref_device, float *out_norm2, float *out_div2) {
  if (!h || !out_norm2 || !out_div2) return HADFL_ERR_INVALID;
  const int rc = hadfl_stats_enqueue(h, ref_device);
  return rc != HADFL_OK ? rc : hadfl_stats_read(h, out_norm2, out_div2);
}

// ---- statistics without any allocation ---------------------------------------------------------
// Fixed scratch in the library image: [0, 256) the completion ticket, then the per-block partial
// sums (2 doubles per block).  In host code the array's name is only a stand-in; the address that
// kernels can use comes from cudaGetSymbolAddress, looked up once per device.
static __device__ __align__(256) unsigned char g_noalloc_scratch[HADFL_NOALLOC_SCRATCH_BYTES];

namespace {
constexpr int kNoallocMaxGpus = 64;
unsigned char *g_noalloc_ptr[kNoallocMaxGpus];  // device address of the scratch, per device
int g_noalloc_sms[kNoallocMaxGpus];
}  // namespace

int hadfl_stats_noalloc(const void *w, int32_t dtype, int32_t n_devices, int64_t n_params,
                        int64_t row_stride_elems, int32_t ref_device, float *out_stats,
                        void *cuda_stream) {
  if (n_devices > HADFL_MAX_DEVICES || n_params > HADFL_NOALLOC_MAX_PARAMS) return HADFL_ERR_TOO_LARGE;
  if (!w || !out_stats || n_devices < 1 || n_params < 1) return HADFL_ERR_INVALID;
  if (dtype != HADFL_DTYPE_FP32 && dtype != HADFL_DTYPE_BF16) return HADFL_ERR_INVALID;
  if (row_stride_elems < n_params || row_stride_elems % 8 != 0) return HADFL_ERR_INVALID;
  if (ref_device < 0 || ref_device >= n_devices) return HADFL_ERR_INVALID;
  if (((uintptr_t)w & 15u) || ((uintptr_t)out_stats & 3u)) return HADFL_ERR_INVALID;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNoallocMaxGpus) return HADFL_ERR_CUDA;
  if (!g_noalloc_ptr[dev]) {  // set-up, once per device, with that device current
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return HADFL_ERR_CUDA;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
      return HADFL_ERR_CUDA;
    g_noalloc_sms[dev] = sms;
    g_noalloc_ptr[dev] = (unsigned char *)p;
  }
  // Both buffers must be device memory of the current device: anything else (a host pointer, another
  // GPU's memory) would turn into a memory fault inside the kernel instead of an error status.
  // cudaPointerGetAttributes allocates nothing.
  {
    const void *ptrs[2] = {w, out_stats};
    for (const void *q : ptrs) {
      cudaPointerAttributes at;
      if (cudaPointerGetAttributes(&at, q) != cudaSuccess) {
        cudaGetLastError();
        return HADFL_ERR_INVALID;
      }
      if ((at.type != cudaMemoryTypeDevice && at.type != cudaMemoryTypeManaged) || at.device != dev)
        return HADFL_ERR_INVALID;
    }
  }
  unsigned int *ticket = (unsigned int *)g_noalloc_ptr[dev];
  double *partials = (double *)(g_noalloc_ptr[dev] + 256);
  // Same grid rule as the handle's statistics launch, capped by what the scratch holds.
  const int64_t lanes = stats_lanes_for(g_noalloc_sms[dev], n_devices, n_params, dtype, HADFL_NOALLOC_MAX_BLOCKS);
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  cudaGetLastError();  // an error left behind by earlier, unrelated work is not this call's
#ifdef HADFL_DEBUG
  // Debug build only: the caller's buffers and the fixed scratch join the table of checked ranges for
  // the duration of the call, which therefore synchronises the device before and after its kernel.
  const size_t es_dbg = dtype == HADFL_DTYPE_BF16 ? 2 : 4;
  cudaDeviceSynchronize();
  debug_add(w, (size_t)n_devices * (size_t)row_stride_elems * es_dbg);
  debug_add(out_stats, sizeof(float) * 2 * (size_t)n_devices);
  debug_add(g_noalloc_ptr[dev], HADFL_NOALLOC_SCRATCH_BYTES);
  debug_publish();
  struct Unregister {
    const void *a, *b, *c;
    ~Unregister() {
      cudaDeviceSynchronize();
      debug_remove(c);
      debug_remove(b);
      debug_remove(a);
      debug_publish();
    }
  } unregister{w, out_stats, g_noalloc_ptr[dev]};
#endif
  // The array keeps the previous call's contents: the ticket must start at zero.
  if (cudaMemsetAsync(ticket, 0, sizeof(unsigned int), stream) != cudaSuccess) return HADFL_ERR_CUDA;
  const unsigned blocks = (unsigned)(lanes * n_devices);
  if (dtype == HADFL_DTYPE_BF16)
    k_stats<__nv_bfloat16, kStatsU><<<blocks, kThreads, 0, stream>>>(
        (const __nv_bfloat16 *)w, row_stride_elems, n_params, n_devices, ref_device, (int)lanes,
        partials, ticket, out_stats);
  else
    k_stats<float, kStatsU><<<blocks, kThreads, 0, stream>>>(
        (const float *)w, row_stride_elems, n_params, n_devices, ref_device, (int)lanes, partials,
        ticket, out_stats);
  return cudaGetLastError() == cudaSuccess ? HADFL_OK : HADFL_ERR_CUDA;
}

int64_t hadfl_stats_grid_lanes(int32_t sm_count, int32_t n_devices, int64_t n_params, int32_t dtype,
                               int64_t max_blocks) {
  if (sm_count < 1 || n_devices < 1 || n_devices > HADFL_MAX_DEVICES || n_params < 1 || max_blocks < 0) return 0;
  if (dtype != HADFL_DTYPE_FP32 && dtype != HADFL_DTYPE_BF16) return 0;
  return stats_lanes_for(sm_count, n_devices, n_params, dtype, max_blocks);
}

int hadfl_read_params(hadfl_handle *h, int32_t id, float *dst, int64_t count) {
  return read_row(h, id, dst, count, false);
}
int hadfl_read_momentum(hadfl_handle *h, int32_t id, float *dst, int64_t count) {
  return read_row(h, id, dst, count, true);
}
int hadfl_write_params(hadfl_handle *h, int32_t id, const float *src, int64_t count) {
  return write_row(h, id, src, count, false);
}
int hadfl_write_momentum(hadfl_handle *h, int32_t id, const float *src, int64_t count) {
  return write_row(h, id, src, count, true);
}

int hadfl_backup_wait(hadfl_handle *h) {
  if (!h) return HADFL_ERR_INVALID;
  if (!h->backup_in_flight) return HADFL_OK;
  DeviceGuard guard(h->device);
  HADFL_CUDA(h, cudaEventSynchronize(h->backup_done));
  h->backup_in_flight = false;
  if (h->cfg.dtype == HADFL_DTYPE_BF16) {
    for (int64_t p = 0; p < h->backup_count; ++p) {
      const uint32_t bits = (uint32_t)h->backup_bf16[(size_t)p] << 16;
      memcpy(h->backup_dst + p, &bits, 4);
    }
  }
  return HADFL_OK;
}

int hadfl_backup_begin(hadfl_handle *h, int32_t device_id, float *dst, int64_t count) {
  if (!h) return HADFL_ERR_INVALID;
  if (!dst || device_id < 0 || device_id >= h->cfg.n_devices || count < 1 || count > h->cfg.n_params)
    return HADFL_ERR_INVALID;
  if (h->backup_in_flight) {  // one backup at a time: finish the previous one first
    const int rc = hadfl_backup_wait(h);
    if (rc != HADFL_OK) return rc;
  }
  DeviceGuard guard(h->device);
  const size_t es = elem_size(h);
  if (!h->backup_stream) {  // first use: staging row, copy stream, two events
    HADFL_CUDA(h, cudaMalloc(&h->d_backup, (size_t)h->cfg.n_params * es));  // copies only: no kernel touches it
    HADFL_CUDA(h, cudaStreamCreateWithFlags(&h->backup_stream, cudaStreamNonBlocking));
    HADFL_CUDA(h, cudaEventCreateWithFlags(&h->backup_ready, cudaEventDisableTiming));
    HADFL_CUDA(h, cudaEventCreateWithFlags(&h->backup_done, cudaEventDisableTiming));
  }
  // Snapshot on the main stream (device to device, ~2 P bytes of HBM traffic), then the slow
  // copy to the host on the copy stream, so that later rounds do not wait for PCIe.
  const char *src = (const char *)h->w + (size_t)device_id * (size_t)h->stride * es;
  HADFL_CUDA(h, cudaMemcpyAsync(h->d_backup, src, (size_t)count * es, cudaMemcpyDeviceToDevice, h->stream));
  HADFL_CUDA(h, cudaEventRecord(h->backup_ready, h->stream));
  HADFL_CUDA(h, cudaStreamWaitEvent(h->backup_stream, h->backup_ready, 0));
  void *host = dst;
  if (h->cfg.dtype == HADFL_DTYPE_BF16) {
    h->backup_bf16.resize((size_t)count);
    host = h->backup_bf16.data();
  }
  HADFL_CUDA(h, cudaMemcpyAsync(host, h->d_backup, (size_t)count * es, cudaMemcpyDeviceToHost, h->backup_stream));
  HADFL_CUDA(h, cudaEventRecord(h->backup_done, h->backup_stream));
  h->backup_in_flight = true;
  h->backup_dst = dst;
  h->backup_count = count;
  return HADFL_OK;
}

int hadfl_get_versions(hadfl_handle *h, uint32_t *versions, uint64_t *step_counts) {
  if (!h) return HADFL_ERR_INVALID;
  for (int i = 0; i < h->cfg.n_devices; ++i) {
    if (versions) versions[i] = h->version[i];
    if (step_counts) step_counts[i] = h->step_count[i];
  }
  return HADFL_OK;
}

int hadfl_set_versions(hadfl_handle *h, const uint32_t *versions, const uint64_t *step_counts) {
  if (!h) return HADFL_ERR_INVALID;
  if (step_counts)
    for (int i = 0; i < h->cfg.n_devices; ++i)
      if (step_counts[i] >> 56) return HADFL_ERR_INVALID;
  for (int i = 0; i < h->cfg.n_devices; ++i) {
    if (versions) h->version[i] = versions[i];
    if (step_counts) h->step_count[i] = step_counts[i];
  }
  return HADFL_OK;
}

int hadfl_set_available(hadfl_handle *h, const uint8_t *mask) {
  if (!h) return HADFL_ERR_INVALID;
  for (int i = 0; i < h->cfg.n_devices; ++i) h->avail[i] = mask ? (mask[i] ? 1 : 0) : 1;
  return HADFL_OK;
}

int hadfl_synchronize(hadfl_handle *h) {
  if (!h) return HADFL_ERR_INVALID;
  DeviceGuard guard(h->device);
  HADFL_CUDA(h, cudaStreamSynchronize(h->stream));
  HADFL_DEBUG_RESULT();
  return HADFL_OK;
}

int hadfl_debug_build(void) {
#ifdef HADFL_DEBUG
  return 1;
#else
  return 0;
#endif
}

int hadfl_debug_check(hadfl_handle *h, uint64_t *out_bad_address) {
  if (!h) return HADFL_ERR_INVALID;
  if (out_bad_address) *out_bad_address = 0;
#ifdef HADFL_DEBUG
  DeviceGuard guard(h->device);
  HADFL_CUDA(h, cudaStreamSynchronize(h->stream));
  if (debug_error(out_bad_address)) return HADFL_ERR_STATE;
#endif
  return HADFL_OK;
}

int hadfl_debug_range_holds(uint64_t lo, uint64_t hi, uint64_t addr, uint64_t nbytes) {
  return range_holds(lo, hi, addr, nbytes) ? 1 : 0;
}

int hadfl_last_cuda_error(const hadfl_handle *h) { return h ? h->last_cuda_error : 0; }
uint64_t hadfl_launch_count(const hadfl_handle *h) { return h ? h->launches : 0; }
int64_t hadfl_row_stride(const hadfl_handle *h) { return h ? h->stride : 0; }
int32_t hadfl_round_grid(const hadfl_handle *h) { return h ? h->round_grid : 0; }

int hadfl_selection_probs(const double *x, const uint8_t *avail, int32_t n, double *out_P) {
  if (!x || !out_P || n < 1 || n > HADFL_MAX_DEVICES) return HADFL_ERR_INVALID;
  return selection_probs(x, avail, n, out_P) ? HADFL_OK : HADFL_ERR_INVALID;
}

int hadfl_selection_draw(const double *x, const uint8_t *avail, int32_t n, int64_t round,
                         uint64_t seed, int32_t k, int32_t *out_selected) {
  if (!x || !out_selected || n < 1 || n > HADFL_MAX_DEVICES) return HADFL_ERR_INVALID;
  return selection_draw(x, avail, n, round, seed, k, out_selected) ? HADFL_OK : HADFL_ERR_INVALID;
}

int hadfl_predict_version(const double *series, int32_t n_obs, double alpha, double m,
                          double *out_prediction) {
  if (!series || !out_prediction || n_obs < 1 || !(alpha > 0.0 && alpha < 1.0)) return HADFL_ERR_INVALID;
  *out_prediction = predict_version(series, n_obs, alpha, m);
  return HADFL_OK;
}

int hadfl_debug_philox(hadfl_handle *h, const uint32_t *counters, const uint32_t *key, int64_t n,
                       uint32_t *out_words) {
  if (!h || !counters || !key || !out_words || n < 0) return HADFL_ERR_INVALID;
  if (n == 0) return HADFL_OK;
  DeviceGuard guard(h->device);
  uint32_t *d_in = nullptr, *d_out = nullptr;
  const size_t bytes = sizeof(uint32_t) * 4 * (size_t)n;
  HADFL_CUDA(h, cudaMalloc((void **)&d_in, bytes));
  cudaError_t e = cudaMalloc((void **)&d_out, bytes);
  if (e == cudaSuccess) e = cudaMemcpyAsync(d_in, counters, bytes, cudaMemcpyHostToDevice, h->stream);
  if (e == cudaSuccess) {
    const PhiloxKeys keys = expand_keys(((uint64_t)key[1] << 32) | key[0]);
    k_debug_philox<<<(unsigned)((n + 255) / 256), 256, 0, h->stream>>>(d_in, keys, n, d_out);
    e = cudaGetLastError();
    ++h->launches;
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(out_words, d_out, bytes, cudaMemcpyDeviceToHost, h->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
  cudaFree(d_in);
  cudaFree(d_out);
  HADFL_CUDA(h, e);
  return HADFL_OK;
}

int hadfl_debug_normals(hadfl_handle *h, int32_t which, const uint32_t *groups, int64_t n,
                        uint64_t step, uint32_t device, float *out_z) {
  if (!h || !groups || !out_z || n < 0 || (which != 0 && which != 1)) return HADFL_ERR_INVALID;
  if (n == 0) return HADFL_OK;
  DeviceGuard guard(h->device);
  uint32_t *d_in = nullptr;
  float4 *d_out = nullptr;
  HADFL_CUDA(h, cudaMalloc((void **)&d_in, sizeof(uint32_t) * (size_t)n));
  cudaError_t e = cudaMalloc((void **)&d_out, sizeof(float4) * (size_t)n);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(d_in, groups, sizeof(uint32_t) * (size_t)n, cudaMemcpyHostToDevice, h->stream);
  if (e == cudaSuccess) {
    const unsigned blocks = (unsigned)((n + 255) / 256);
    if (which == 0)
      k_debug_normals<NormalsFast><<<blocks, 256, 0, h->stream>>>(
          d_in, n, (uint32_t)step, device, kTagGrad | ((uint32_t)(step >> 32) & 0xFFFFFFu), h->keys, d_out);
    else
      k_debug_normals<NormalsAccurate><<<blocks, 256, 0, h->stream>>>(d_in, n, 0u, 0u, kTagInit,
                                                                       h->keys, d_out);
    e = cudaGetLastError();
    ++h->launches;
  }
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(out_z, d_out, sizeof(float4) * (size_t)n, cudaMemcpyDeviceToHost, h->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
  cudaFree(d_in);
  cudaFree(d_out);
  HADFL_CUDA(h, e);
  return HADFL_OK;
}

}  // extern "C"
