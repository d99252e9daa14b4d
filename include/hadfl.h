/*
 * hadfl.h - C ABI of the HADFL round hot path on one NVIDIA B200 (sm_100a).
 *
 * The method is HADFL (Cao et al., "HADFL: Heterogeneity-aware Decentralized Federated Learning
 * Framework", arXiv 2111.08274).  N simulated heterogeneous devices each hold a flat parameter
 * vector w (fp32, or bf16 storage) and a momentum vector m (fp32, or bf16 storage next to bf16
 * parameters).  All replicas live in one
 * device-memory arena: row i of w is device i's model, at w_ptr + i * row_stride_elems elements.
 *
 * One training round is the call sequence
 *     hadfl_local_step   every device runs its own number E_i of local SGD steps
 *                        (Eq. 3; Algorithm 1, "for e_k = 0 to E_k")
 *     hadfl_select       N_p devices are drawn with the probability-based selection function
 *                        (Eq. 8; Section "Heterogeneity-aware training strategy generation")
 *     hadfl_aggregate    the selected replicas are averaged and the average is written back to
 *                        them (Eq. 5; Algorithm 1, "partial synchronization")
 *     hadfl_stats        per-replica squared norm and squared distance to a reference replica
 *                        (diagnostics; not in the paper)
 * or the single call hadfl_round, which runs that whole sequence in one kernel with identical
 * results; and, when a model is wanted on the host (the coordinator's model backup, Section
 * "Overall Design" item 9), hadfl_read_params or the overlapped hadfl_backup_begin / _wait.
 *
 * General rules
 *   - Every function returns an int status: HADFL_OK, HADFL_ERR_INVALID (bad argument, duplicate or
 *     out-of-range device id, k larger than the number of available devices, ...), HADFL_ERR_CUDA
 *     (a CUDA call failed: hadfl_last_cuda_error gives the cudaError_t value), HADFL_ERR_STATE
 *     (call not valid in the handle's state).  Nothing aborts and no kernel traps.  After
 *     HADFL_ERR_INVALID the handle and the arena are unchanged.
 *   - Pointer arguments are HOST pointers unless the comment says "device".  The caller owns every
 *     buffer it passes; the library has copied what it needs when the call returns.
 *   - All device work is enqueued on the one stream given at hadfl_init.  Calls return without
 *     waiting for the GPU, except those marked "synchronises", which wait for that stream.
 *   - A handle is not thread-safe.
 *   - The synthetic gradient of parameter p of device i at its local step s is
 *     grad_std * z, z a standard normal obtained by Box-Muller from the Philox4x32-10 block with
 *     key = seed and counter = (p / 4, s mod 2^32, i, 'G' << 24 | s >> 32); lane p mod 4 of the
 *     block.  It replaces forward/backward propagation, which is outside this library.
 */
#ifndef HADFL_H_
#define HADFL_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HADFL_OK 0
#define HADFL_ERR_INVALID 1
#define HADFL_ERR_CUDA 2
#define HADFL_ERR_STATE 3
#define HADFL_ERR_TOO_LARGE 4 /* only hadfl_stats_noalloc: the problem exceeds its fixed scratch */

#define HADFL_MAX_DEVICES 32 /* largest N, and therefore largest k */

#define HADFL_DTYPE_FP32 0 /* w stored as fp32 */
#define HADFL_DTYPE_BF16 1 /* w stored as bf16, all arithmetic in fp32, one rounding per call */

/* How the local update rounds what it stores as bf16 (once per call and value).  Not in the paper,
 * which trains in fp32: with nearest-even storage an update below half a bf16 spacing is lost
 * every time, with stochastic storage it survives on average.  Stochastic: the 16 random bits r are
 * added to the fp32 bit pattern and the low 16 bits dropped, so a finite value moves to its
 * neighbour of larger magnitude with probability (dropped bits) / 2^16 (infinities and NaNs are
 * rounded to nearest).  r comes from the Philox4x32-10 block with key = seed and counter
 * (p / 4, s mod 2^32, i, 'R' << 24 | s >> 32), s the index of the LAST step the call runs on device
 * i: lane p mod 4 of the block, low half for the parameter, high half for the momentum. */
#define HADFL_ROUND_NEAREST 0
#define HADFL_ROUND_STOCHASTIC 1

#define HADFL_WEIGHTS_UNIFORM 0 /* a_j = 1/k: Eq. 5 with K read as the number of selected devices */
#define HADFL_WEIGHTS_VERSION 1 /* extension, not in the paper: a_j proportional to f(v_j) of Eq. 8 */

typedef struct hadfl_handle hadfl_handle;

typedef struct hadfl_config {
  int32_t n_devices;        /* N, 1..HADFL_MAX_DEVICES */
  int64_t n_params;         /* P >= 1, P <= 2^34 - 4 */
  int32_t dtype;            /* HADFL_DTYPE_* */
  float momentum;           /* mu of the local update */
  float weight_decay;       /* wd of the local update */
  float grad_std;           /* standard deviation of the synthetic gradients, >= 0 */
  float init_std;           /* standard deviation of the initial model */
  uint64_t seed;            /* key of the counter-based generator */
  double version_scale;     /* versions are multiplied by this before Eq. 8 (1.0 = the paper) */
  int32_t weight_mode;      /* HADFL_WEIGHTS_* */
  void *w_ptr;              /* DEVICE pointer to the parameter arena, or NULL: the library
                               allocates it (and the momentum arena) and frees it at destroy */
  void *m_ptr;              /* DEVICE pointer to the momentum arena (fp32, or bf16 per m_dtype);
                               NULL iff w_ptr is NULL */
  int64_t row_stride_elems; /* elements between rows; 0 = P rounded up to a multiple of 32.
                               Must be >= P and a multiple of 8.  Caller-owned arenas must be
                               16-byte aligned, hold N * row_stride_elems elements each and outlive
                               the handle. */
  void *cuda_stream;        /* cudaStream_t on which all work is enqueued (NULL = default stream) */
  int32_t m_dtype;          /* HADFL_DTYPE_* of the momentum; bf16 only together with bf16 parameters */
  int32_t rounding;         /* HADFL_ROUND_* of the local update's bf16 stores; stochastic only with
                               bf16 parameters.  Aggregation and global synchronisation always round
                               to nearest even. */
} hadfl_config;

/* Algorithm 1, step 1 ("synchronize the initial models"): creates the handle on the current CUDA
 * device, fills every row of w with the same w_(0)[p] = init_std * z(seed, p) and m with zeros
 * (padding between rows too), and sets all versions and step counters to 0.  Asynchronous.
 * On HADFL_ERR_CUDA *out is still a handle (so that the error code can be read) and must be
 * destroyed; on other errors *out is NULL. */
int hadfl_init(const hadfl_config *config, hadfl_handle **out);

/* Waits for the stream, frees what the library allocated.  NULL is accepted. */
int hadfl_destroy(hadfl_handle *h);

/* Local update, Eq. 3 / Algorithm 1 (heterogeneity-aware local steps E_k): device device_ids[j]
 * runs steps[j] >= 0 SGD steps on its own replica, in ONE kernel launch for all listed devices:
 *     g = fma(wd, w, grad_std * z);  m = fma(mu, m, g);  w = fma(-lr, m, w)
 * (momentum and weight decay follow the PyTorch SGD convention; Eq. 3 is mu = wd = 0).  w and m
 * are read and written once per call whatever the step count; values stored as bf16 are widened on
 * entry, kept in fp32 through the steps and rounded once at the end (per config.rounding).  A device
 * listed with 0 steps is not touched.  Afterwards the version and the step counter of each listed
 * device have grown by its step count.
 * device_ids: n distinct ids in [0, N); 1 <= n <= N.  Asynchronous. */
int hadfl_local_step(hadfl_handle *h, const int32_t *device_ids, const int32_t *steps, int32_t n,
                     float lr);

/* Probability-based selection, Eq. 8: P(i) = f(x_i) / sum_n f(x_n) over the available devices,
 * x_i = versions[i] * version_scale, f the unit-variance Gaussian density about mu, mu the third
 * quartile (linear interpolation) of the available x.  k distinct devices are drawn one after the
 * other, each with probability proportional to f among those not yet drawn (uniformly if all
 * remaining f underflow); out_selected receives them in draw order, which is also the ring order
 * and the summation order of hadfl_aggregate.  The random stream is Philox4x32-10 keyed by `seed`
 * with counter (t, 0, round, 'S' << 24): the result is a pure function of the arguments, the
 * availability mask and version_scale.
 * versions: N doubles, or NULL for the handle's own counters.  Host only; no GPU work. */
int hadfl_select(hadfl_handle *h, int64_t round, const double *versions, uint64_t seed, int32_t k,
                 int32_t *out_selected);

/* Eq. 8 itself: out_P[i] = P(i) (0 for unavailable devices).  Host only. */
int hadfl_select_probs(hadfl_handle *h, const double *versions, double *out_P);

/* Eq. 8 on the versions the devices WILL have once device_ids[j] has run steps[j] more local steps
 * (each listed device's version grows by its step count; the others keep theirs): the probabilities
 * from which hadfl_round(device_ids, steps, ..., versions = NULL) draws its selection, for callers
 * that want to log them beside a fused round.  n distinct ids, steps >= 0.  Host only. */
int hadfl_select_probs_after(hadfl_handle *h, const int32_t *device_ids, const int32_t *steps, int32_t n,
                             double *out_P);

/* Partial aggregation, Eq. 5 / Algorithm 1 "partial synchronization", fused with the write-back:
 *     acc = a_0 * w[selected[0]];  acc = fma(a_j, w[selected[j]], acc), j = 1..k-1;
 *     w[selected[j]] = acc for all j          (one kernel, every element touched once)
 * a_j = 1/k, or the version-dependent weights of weight_mode 1 computed from `versions` (N doubles,
 * NULL = the handle's counters).  Momentum is not touched.  Afterwards every selected device carries
 * the largest version among them.  selected: k distinct ids, 1 <= k <= N.  Asynchronous. */
int hadfl_aggregate(hadfl_handle *h, const int32_t *selected, int32_t k, const double *versions);

/* The weights a_j that hadfl_aggregate would use (out_a: k floats).  Host only. */
int hadfl_aggregation_weights(hadfl_handle *h, const int32_t *selected, int32_t k,
                              const double *versions, float *out_a);

/* Global synchronisation, Algorithm 1 "send w to devices whose Flag = 0": the parameters of
 * device src overwrite those of the n devices dst_ids (distinct, none equal to src, n may be 0),
 * which also take its version.  One kernel: one read and n writes per element.  Asynchronous. */
int hadfl_broadcast(hadfl_handle *h, int32_t src, const int32_t *dst_ids, int32_t n);

/* Global synchronisation read as a mix.  Section "Model aggregation and fault-tolerant" says that an
 * unselected device folds the model it receives into its own parameters before its next local
 * steps, without giving a formula; Algorithm 1 simply sends the model.  hadfl_broadcast is the
 * second reading (overwrite), this call the first, as a convex combination with weight beta on the
 * received model:
 *     w[dst] = fma(beta, w[src], (1 - beta) * w[dst])      (1 - beta and the product rounded to fp32)
 * for each of the n devices dst_ids (distinct, none equal to src, n may be 0); 0 <= beta <= 1.
 * beta = 1 gives the overwrite, beta = 0 leaves the receivers as they are.  bf16 storage is rounded
 * to nearest even.  Momentum is not touched.  A receiver's version becomes the larger of its own and
 * the sender's (the sender's when beta = 1).  One kernel: 1 + n reads and n writes per element.
 * Asynchronous. */
int hadfl_integrate(hadfl_handle *h, int32_t src, const int32_t *dst_ids, int32_t n, float beta);

/* Which reading hadfl_round's global synchronisation (sync_all != 0) takes: beta = 1 (the default)
 * is the overwrite of hadfl_broadcast, 0 <= beta < 1 the mix of hadfl_integrate with that weight.
 * Host only. */
int hadfl_set_sync_beta(hadfl_handle *h, float beta);

/* One whole round in ONE kernel: Algorithm 1's local steps of every listed device (Eq. 3), the
 * selection (Eq. 8), the partial aggregation with write-back (Eq. 5), optionally the global
 * synchronisation (Algorithm 1, "send w to devices whose Flag = 0": sync_all != 0 sends the
 * aggregate to every other device) and the statistics with the aggregate as reference.  It is
 * exactly the sequence
 *     hadfl_local_step(device_ids, steps, n, lr); hadfl_select(round, versions, seed, k);
 *     hadfl_aggregate(selected, k, versions);
 *     [hadfl_broadcast(selected[0], all others); or hadfl_integrate(..., beta), see hadfl_set_sync_beta]
 *     hadfl_stats_enqueue(selected[0])
 * - same parameters, momentum, versions and step counters, bit for bit - but each parameter and
 * momentum value is read and written once: the aggregate is formed in registers from the freshly
 * updated replicas and never re-read.  This is possible because selection depends on versions only,
 * and the versions after the local steps are known before they run (versions == NULL uses them;
 * a caller-supplied array is used as given).  The statistics are summed in a different (equally
 * fixed) order than hadfl_stats_enqueue does, so they agree with it to rounding, not bit for bit;
 * read them with hadfl_stats_read.  out_selected: k ids in draw order.  Devices not listed run no
 * steps.  Asynchronous. */
int hadfl_round(hadfl_handle *h, const int32_t *device_ids, const int32_t *steps, int32_t n, float lr,
                int64_t round, const double *versions, uint64_t seed, int32_t k, int32_t sync_all,
                int32_t *out_selected);

/* A run of consecutive rounds enqueued by one call (the coordinator's loop of Algorithm 1 over the
 * synchronisation rounds, for callers whose per-call overhead would otherwise bound small models):
 * for i = 0 .. n_rounds-1, round r = first_round + i is exactly
 *     hadfl_round(all N devices in id order, steps + i * N, N, lr, r, NULL, seed, k,
 *                 sync_every > 0 && (r + 1) % sync_every == 0, out_selected + i * k)
 * steps: n_rounds x N step counts; out_selected: n_rounds x k ids, or NULL.  Stops at the first
 * round that fails and returns its status (earlier rounds stay enqueued).  Asynchronous.  (Hundreds of
 * launches queued at once were measured 1-3 % slower per round on large models than a queue a few
 * launches deep: enqueue long runs in pieces.) */
int hadfl_rounds(hadfl_handle *h, int64_t first_round, int32_t n_rounds, const int32_t *steps, float lr,
                 uint64_t seed, int32_t k, int32_t sync_every, int32_t *out_selected);

/* Rounds per launch.  Every operation of a round (Eq. 3, Eq. 5, the send to the other devices) is
 * elementwise in the parameter index, and the selections (Eq. 8) depend on versions the host knows
 * beforehand, so hadfl_rounds may hand several consecutive rounds to ONE launch of the fused kernel:
 * a block takes its columns through all of them before it moves to the next columns, and from the
 * second round on the replicas are read from L2 instead of HBM.  Results - parameters, momentum,
 * counters, selections - are those of the rounds launched one by one, bit for bit; so are every
 * round's statistics, except that batches on large fp32 arenas whose devices run at most 1.5 steps
 * on average are taken in packs of half the width, which sums the statistics in a different
 * (equally fixed) order: they then agree to rounding.  hadfl_rounds batches the rounds that gain from it (every device runs at most two
 * steps and rounding is to nearest even, or the whole arena - parameters and momentum of all
 * devices - is at most 64 MiB) and launches the others singly.
 * hadfl_set_round_batch: the most rounds per launch, 1 .. 8 (default 8; 1 = never batch);
 * HADFL_ERR_INVALID outside that range.  hadfl_round_batch returns the setting (0 for NULL). */
int hadfl_set_round_batch(hadfl_handle *h, int32_t max_rounds);
int32_t hadfl_round_batch(const hadfl_handle *h);
/* Columns per thread (8, or 4 for the half-width packs above) in the most recent launch of the fused
 * round kernel; 0 before the first one or for NULL.  For tests and logs. */
int32_t hadfl_last_round_pack(const hadfl_handle *h);

/* The statistics that the fused kernel left for the round `back` rounds before the last one of its
 * most recent launch (back = 0: the last round, the same as hadfl_stats_read).  A launch keeps the
 * statistics of each of its rounds; HADFL_ERR_STATE when `back` reaches beyond the rounds of that
 * launch or no fused round has run.  Synchronises the stream. */
int hadfl_stats_read_round(hadfl_handle *h, int32_t back, float *out_norm2, float *out_div2);

/* Per-replica statistics (not in the paper; diagnostics of how far the replicas have drifted):
 * out_norm2[i] = sum_p w_i[p]^2, out_div2[i] = sum_p (w_i[p] - w_ref[p])^2, N floats each.
 * Deterministic: fixed grid, fixed summation order, fp32 within a chunk, fp64 above.
 * hadfl_stats = enqueue + read; hadfl_stats_read synchronises and returns the last enqueued result. */
int hadfl_stats_enqueue(hadfl_handle *h, int32_t ref_device);
int hadfl_stats_read(hadfl_handle *h, float *out_norm2, float *out_div2);
int hadfl_stats(hadfl_handle *h, int32_t ref_device, float *out_norm2, float *out_div2);

/* Statistics for callers that must not allocate device memory.  (The paper has no counterpart: this
 * is the computation of hadfl_stats behind an entry point with a different memory contract.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a process whose whole device
 * memory has been handed to another allocator or is budgeted to the last byte, in a latency-critical
 * loop that cannot afford the device-wide synchronisation an allocation implies, or in a component
 * that is simply not allowed to own device memory.  Such a caller cannot even create a handle,
 * because hadfl_init allocates the scratch of the statistics kernel.  This entry point therefore
 * takes no handle and calls no cudaMalloc, cudaFree or any other allocating routine: its scratch
 * (per-block partial sums and the completion ticket) lives in a fixed array of
 * HADFL_NOALLOC_SCRATCH_BYTES inside the library image, which every GPU that loads the library
 * holds until the process exits.
 *
 *   w            DEVICE pointer, 16-byte aligned, to N rows of row_stride_elems elements
 *                (fp32 or bf16 per dtype) on the CURRENT device; read only.
 *   out_stats    DEVICE pointer to 2N floats on the same device: norm2[0..N) then div2[0..N),
 *                written by the kernel; valid once work enqueued on `cuda_stream` has completed.
 *   cuda_stream  cudaStream_t the work is enqueued on.  Asynchronous.
 *
 * Limits: 1 <= n_devices <= HADFL_MAX_DEVICES and 1 <= n_params <= HADFL_NOALLOC_MAX_PARAMS;
 * anything larger returns HADFL_ERR_TOO_LARGE and enqueues nothing.  Other bad arguments (NULL or
 * misaligned pointers, a w or out_stats that is not device memory of the current device - checked
 * with cudaPointerGetAttributes, so that a host pointer or another GPU's buffer is refused here
 * instead of faulting in the kernel -, stride < n_params or not a multiple of 8, ref_device out of
 * range) return HADFL_ERR_INVALID; a failing CUDA call returns HADFL_ERR_CUDA (an error left behind
 * by earlier, unrelated CUDA work is cleared first and not reported).
 *
 * The first call on each device looks up the device address of the scratch array (once per
 * device); make that first call outside any stream capture and from one thread only.  All calls on a device share the one
 * array, which still holds what the previous call left there: each call re-zeroes the ticket on
 * the stream before its kernel, and two calls whose kernels overlap on the GPU (different streams,
 * no ordering between them) race on the scratch and give wrong sums - order them.  The result
 * equals hadfl_stats for the same arena bit for bit when the grids agree, and within the same
 * 1e-5 relative bound otherwise. */
#define HADFL_NOALLOC_MAX_BLOCKS 2048
#define HADFL_NOALLOC_SCRATCH_BYTES (256 + 2 * 8 * HADFL_NOALLOC_MAX_BLOCKS)
#define HADFL_NOALLOC_MAX_PARAMS (((int64_t)1 << 31) - 4)
int hadfl_stats_noalloc(const void *w, int32_t dtype, int32_t n_devices, int64_t n_params,
                        int64_t row_stride_elems, int32_t ref_device, float *out_stats,
                        void *cuda_stream);

/* The grid rule of the statistics kernel, as a pure host function (no GPU): blocks per row for a GPU
 * with sm_count SMs - one wave of 8 blocks per SM split evenly over the n_devices rows, at most one
 * block per 16 KB chunk of a row, and, when max_blocks > 0 (hadfl_stats_noalloc passes
 * HADFL_NOALLOC_MAX_BLOCKS), at most max_blocks blocks in all.  Returns 0 for invalid arguments.
 * With 148 SMs the cap of 2048 blocks is never reached (8 * 148 = 1184 resident blocks); it takes
 * a GPU of more than 256 SMs. */
int64_t hadfl_stats_grid_lanes(int32_t sm_count, int32_t n_devices, int64_t n_params, int32_t dtype,
                               int64_t max_blocks);

/* Model backup (Section "Overall Design", item 9) and checkpointing.  `count` elements starting at
 * parameter 0 of device_id; bf16 storage (of parameters or momentum) is widened to / rounded from
 * fp32 (nearest even).
 * Reads synchronise; writes are ordered on the stream and have consumed src on return. */
int hadfl_read_params(hadfl_handle *h, int32_t device_id, float *dst, int64_t count);
int hadfl_read_momentum(hadfl_handle *h, int32_t device_id, float *dst, int64_t count);
int hadfl_write_params(hadfl_handle *h, int32_t device_id, const float *src, int64_t count);
int hadfl_write_momentum(hadfl_handle *h, int32_t device_id, const float *src, int64_t count);

/* Model backup that overlaps with the rounds that follow (Section "Overall Design", item 9: the model
 * manager "regularly fetches the latest model").  hadfl_backup_begin takes a snapshot of the first
 * `count` parameters of device_id as they are at this point of the handle's stream (one device-to-
 * device copy on that stream into a staging row the library allocates on first use) and then moves
 * it to `dst` on a separate copy stream: the caller and the later work on the handle's stream do not
 * wait for the transfer.  dst (fp32, widened from bf16 storage) must stay valid until
 * hadfl_backup_wait returns, which blocks until the data has arrived; use pinned host memory for the
 * copy to be asynchronous.  One backup is in flight per handle: a second hadfl_backup_begin first
 * waits for the previous one.  hadfl_backup_wait without a backup in flight returns HADFL_OK. */
int hadfl_backup_begin(hadfl_handle *h, int32_t device_id, float *dst, int64_t count);
int hadfl_backup_wait(hadfl_handle *h);

/* Versions v_i ("actual parameter version of device i", Section "Runtime information prediction")
 * and per-device step counters (the index into each device's gradient stream).  N entries each;
 * either pointer may be NULL.  Restoring w, m, versions and step counters resumes a run exactly. */
int hadfl_get_versions(hadfl_handle *h, uint32_t *versions, uint64_t *step_counts);
int hadfl_set_versions(hadfl_handle *h, const uint32_t *versions, const uint64_t *step_counts);

/* The set of available devices N_avl over which Eq. 8 normalises (liveness monitor, Section
 * "Overall Design" item 1).  mask: N bytes, non-zero = available; NULL = all. */
int hadfl_set_available(hadfl_handle *h, const uint8_t *mask);

/* Waits for the handle's stream. */
int hadfl_synchronize(hadfl_handle *h);

/* cudaError_t value of the last failed CUDA call on this handle (0 if none). */
int hadfl_last_cuda_error(const hadfl_handle *h);

/* Number of kernels this handle has launched so far. */
uint64_t hadfl_launch_count(const hadfl_handle *h);

/* Row stride, in elements, of the handle's arenas. */
int64_t hadfl_row_stride(const hadfl_handle *h);

/* Number of thread blocks one hadfl_round launch of this handle uses (diagnostics; each block works
 * on chunks of 2048 consecutive parameters of every device). */
int32_t hadfl_round_grid(const hadfl_handle *h);

/* ---- host-only functions (no handle, no GPU) ------------------------------------------------- */

/* Eq. 8 on plain arrays: x (n doubles, already scaled), avail (n bytes or NULL), out_P (n). */
int hadfl_selection_probs(const double *x, const uint8_t *avail, int32_t n, double *out_P);

/* The draw of hadfl_select on plain arrays. */
int hadfl_selection_draw(const double *x, const uint8_t *avail, int32_t n, int64_t round,
                         uint64_t seed, int32_t k, int32_t *out_selected);

/* Runtime version prediction, Eq. 7 (Brown's double exponential smoothing, 0 < alpha < 1):
 * v1_j = alpha v_j + (1-alpha) v1_{j-1}, v2_j = alpha v1_j + (1-alpha) v2_{j-1}, both started at
 * v_0; prediction m rounds after the last observation = (2 v1 - v2) + alpha/(1-alpha) (v1 - v2) m.
 * series: n_obs >= 1 observed versions of one device.  Feeds the `versions` argument of
 * hadfl_select when the coordinator plans with predicted instead of actual versions. */
int hadfl_predict_version(const double *series, int32_t n_obs, double alpha, double m,
                          double *out_prediction);

/* ---- the debug build ---------------------------------------------------------------------------
 * libhadfl_debug.so is this library compiled with -DHADFL_DEBUG: every access a kernel makes to the
 * arenas and every store to the library's scratch buffers is first checked against the device
 * address ranges the handle registered.  An access outside them is skipped (loads read zeros) and
 * recorded; no kernel traps or asserts; and every call marked "synchronises" (and
 * hadfl_synchronize) then returns HADFL_ERR_STATE.  It stands in for a memory checker.  One GPU
 * per process; slower (a table lookup per access; hadfl_init, hadfl_destroy and
 * hadfl_stats_noalloc synchronise the device).  Results are identical to the normal build. */

/* 1 in the debug build, 0 otherwise. */
int hadfl_debug_build(void);

/* Waits for the handle's stream; debug build: HADFL_ERR_STATE if any kernel so far skipped an
 * out-of-range access (*out_bad_address, if not NULL, receives the first such device address);
 * normal build: HADFL_OK. */
int hadfl_debug_check(hadfl_handle *h, uint64_t *out_bad_address);

/* The predicate the debug build applies on the device, as a host function: 1 if the byte range
 * [addr, addr + nbytes) lies inside [lo, hi), else 0 (no arithmetic in it can overflow). */
int hadfl_debug_range_holds(uint64_t lo, uint64_t hi, uint64_t addr, uint64_t nbytes);

/* ---- diagnostics of the on-device generator (used by the tests) -------------------------- */

/* Philox4x32-10 on the GPU: counters (n x 4 words), key (2 words) -> out_words (n x 4).
 * Host pointers; allocates temporaries; synchronises. */
int hadfl_debug_philox(hadfl_handle *h, const uint32_t *counters, const uint32_t *key, int64_t n,
                       uint32_t *out_words);

/* The normals the local-update kernel draws for device `device` at step `step` for the n column
 * groups `groups` (out_z: n x 4 floats), and (which = 1) those of the initial model.
 * Host pointers; allocates temporaries; synchronises. */
int hadfl_debug_normals(hadfl_handle *h, int32_t which, const uint32_t *groups, int64_t n,
                        uint64_t step, uint32_t device, float *out_z);

#ifdef __cplusplus
}
#endif
#endif /* HADFL_H_ */
