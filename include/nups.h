/*
 * nups.h - C ABI of a single-GPU parameter store with non-uniform (skew-aware)
 * parameter access, after NuPS (arXiv 2104.00501).
 *
 * The store keeps one fp32 value row per key in device memory (optionally a
 * second "accumulator" row for AdaGrad), serves pull (row gather) and push
 * (additive scatter) by key, manages hot keys by replication and the rest in
 * place, and draws sampling accesses inside the store under the paper's four
 * conformity levels.
 *
 * Conventions for every call below
 *   - `nups_store*` is an opaque host object owned by the library.
 *   - Arguments named d_* are DEVICE pointers owned by the caller; the library
 *     reads or writes them only in stream order of the call and keeps no
 *     reference afterwards.  Arguments named h_* are HOST pointers.  Everything
 *     else is passed by value.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls enqueue work on it and return; results are ready when the stream
 *     reaches that point.  Calls that return a value through an h_* pointer
 *     synchronise the stream first and say so.
 *   - Keys are uint32 in [0, num_keys).  A key outside the range is never
 *     dereferenced: the access is skipped (a pulled row is zero-filled) and the
 *     device status word is set to NUPS_EKEY; nups_status_check reports it.
 *   - Rows hold `value_len` values, contiguous; a row must be a multiple of 16
 *     bytes (value_len a multiple of 4 for fp32 values, of 2 for fp64 values).
 *   - Value type: fp32 unless the store was created with value_bytes = 8.  Then
 *     both tables, the replicas and every value buffer that crosses this
 *     interface (the void* arguments of pull, push, table_copy, pull_sample)
 *     hold doubles; additions are done in double; nups_step_complex and
 *     nups_step_mf compute in double.  fp32 only: nups_step_sgns / nups_run_sgns,
 *     nups_step_mf_by_column, clip_factor, sync_period_us,
 *     nups_probe_reduction_rate (NUPS_ESTATE or NUPS_EINVAL otherwise).
 *   - Item i of a call over n items belongs to logical worker
 *     q(i) = floor(i * workers / n) (contiguous chunks).  Workers stand for the
 *     paper's nodes: each has its own replica of every replicated key and its
 *     own sample stream.
 *   - Return value: NUPS_OK or a negative nups_status.  Host-detectable errors
 *     are returned at once and enqueue nothing.
 *   - The library's calls on one store are not thread-safe.
 */
#ifndef NUPS_H
#define NUPS_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct nups_store nups_store;
typedef int64_t nups_handle;
typedef int32_t nups_status;

enum {
    NUPS_OK = 0,
    NUPS_EINVAL = -1,  /* bad argument                                              */
    NUPS_ENOMEM = -2,  /* device or host allocation failed, or a table is full       */
    NUPS_ECUDA = -3,   /* a CUDA runtime call failed; see nups_last_cuda_error       */
    NUPS_EKEY = -4,    /* a key >= num_keys was seen on the device (access skipped)  */
    NUPS_ESTATE = -5,  /* over-pull of a handle, level needs ownership tracking, ... */
    NUPS_ETIMEOUT = -6 /* a bounded device-side wait gave up                         */
};
enum { NUPS_SINGLE = 0, NUPS_REPLICATE = 1 };
enum { NUPS_CONFORM = 1, NUPS_BOUNDED = 2, NUPS_LONGTERM = 3, NUPS_NONCONFORM = 4 };

/* Creation-time settings.  Zero-initialise, then set what differs; a NULL config
 * means all defaults.                                                           */
typedef struct nups_config {
    uint32_t workers;         /* R logical workers, 1..254; 0 = default 8                     */
    uint32_t sync_interval;   /* nups_step_* merges replicas every this many steps;           */
                              /* 0 = never automatically                                      */
    uint32_t deterministic;   /* 1: pushes are applied in item order per destination row      */
                              /*    (sort + ordered reduction; reproducible);                 */
                              /* 0: atomic adds in any order (fast)                           */
    uint32_t with_adagrad;    /* 1: allocate the accumulator table                            */
    uint32_t count_accesses;  /* 1: every pulled, pushed or sampled key adds 1 to its count   */
    uint32_t track_ownership; /* 1: keep the key -> owning worker map that LONG-TERM and      */
                              /*    NON-CONFORM sampling need                                 */
    uint32_t smem_hot_rows;   /* fast mode: hot slots below this number are accumulated in    */
                              /*    shared memory inside a kernel before reaching the         */
                              /*    worker's replica; 0 = library default                     */
    uint32_t sync_period_us;  /* > 0: a background thread merges the replicas every this many  */
                              /*    microseconds, see nups_set_sync_period; fast mode only    */
    float    clip_factor;     /* > 0: nups_step_sgns and nups_step_mf clip every update to a   */
                              /*    replicated key at clip_factor times the mean norm of such  */
                              /*    updates so far, see nups_get_clip_stats; 0 = no clipping   */
    uint32_t max_device_mib;  /* > 0: the store never holds more than this many MiB of device memory (tables,   */
                              /*    maps, replicas, alias tables, handles, scratch); a call that would need    */
                              /*    more returns NUPS_ENOMEM before it allocates anything and changes nothing  */
    uint32_t first_epoch;     /* number from which calls that move keys are counted (24 bits, wraps; see        */
                              /*    track_ownership); only of interest to tests of the wrap-around              */
    uint32_t merge_mean;      /* 1: a merge adds the MEAN of the pending updates of the workers that touched a  */
                              /*    replicated key since the last merge instead of their sum (damps the summed  */
                              /*    duplicate updates of very frequent keys); not with sync_period_us           */
    uint32_t value_bytes;     /* 0 or 4: fp32 values; 8: fp64 values (Table 2: the knowledge-graph and matrix-  */
                              /*    factorization tasks use 8-byte values), see "Value type" above              */
    uint32_t reserved[3];
} nups_config;

/* ---- store (Section 3.1: keys, pull, push) -------------------------------- */

/* Allocate a store of num_keys rows of value_len floats, zero-filled, no key
 * replicated.  *h_out receives the store.  NUPS_EINVAL: num_keys == 0 or
 * > 2^32-1, value_len == 0 or rows not a multiple of 16 bytes, workers > 254,
 * value_bytes other than 0, 4, 8, or 8 together with clip_factor or
 * sync_period_us.  NUPS_ENOMEM:
 * the device has not enough memory, or the store's own limit (max_device_mib) is
 * smaller than what the tables and maps need; that limit is checked before the
 * device is touched.                                                           */
nups_status nups_create(uint64_t num_keys, uint32_t value_len, const nups_config* h_cfg, nups_store** h_out);

/* Free everything the store owns.  Synchronises the device.                   */
nups_status nups_destroy(nups_store* store);

/* Device pointer of the value (which = 0) or accumulator (which = 1) table,
 * row-major [num_keys][row_stride_values].  The caller may read or write it in
 * stream order (e.g. to load start values); rows of replicated keys do not
 * include updates that are still pending in replicas.                         */
nups_status nups_table_ptr(nups_store* store, int which, void** h_ptr, uint64_t* h_row_stride_values);

/* Copy a whole table between the store and a caller buffer d_buf of
 * num_keys * value_len values, in stream order: to_store = 1 loads start values
 * into the table, to_store = 0 takes a snapshot of it.                         */
nups_status nups_table_copy(nups_store* store, int which, void* d_buf, int to_store, void* stream);

/* Fill a table with seeded start values: element e gets
 * (int(bits 8..31 of word e mod 4 of Philox4x32-10(counter = (e/4, 0, which, 3),
 *  key = seed)) - 2^23) * (scale * 2^-23), uniform in [-scale, scale).         */
nups_status nups_init_uniform(nups_store* store, int which, uint64_t seed, float scale, void* stream);

/* pull (Section 3.1): d_out[i][:] = current value of d_keys[i] as worker q(i)
 * sees it: the stored row, plus the worker's own pending replica updates when
 * the key is replicated (Section 3.2).  d_out is [n][value_len].
 * nups_pull2 also returns the accumulator rows (either output may be NULL).   */
nups_status nups_pull(nups_store* store, const uint32_t* d_keys, uint64_t n, void* d_out, void* stream);
nups_status nups_pull2(nups_store* store, const uint32_t* d_keys, uint64_t n, void* d_out_val, void* d_out_acc,
                       void* stream);

/* push (Section 3.1; replica accumulation Section 3.1.2): add d_delta[i][:] to
 * the row of d_keys[i], every duplicate applied.  Updates to a replicated key
 * go to worker q(i)'s replica and reach the stored row at the next nups_sync.
 * deterministic = 1: per destination row the deltas are added one by one in
 * ascending i.  nups_push2 updates both tables from one call (AdaGrad state
 * lives beside the value, Section 5.1 / Table 2); either delta may be NULL.   */
nups_status nups_push(nups_store* store, const uint32_t* d_keys, uint64_t n, const void* d_delta, void* stream);
nups_status nups_push2(nups_store* store, const uint32_t* d_keys, uint64_t n, const void* d_delta_val,
                       const void* d_delta_acc, void* stream);

/* Ordered push for callers that must not allocate device memory while they run:
 * code between the start and end of a latency-critical serving loop, a process
 * whose memory pool was handed out in full at start-up, or a host thread that
 * may not take the allocator's device-wide synchronisation.  (The paper has no
 * counterpart; nups_push in deterministic mode sorts the rows by destination and
 * may grow the store's scratch buffer with cudaMalloc/cudaFree when a call is
 * larger than any before it.)  This variant does the same work with its sort
 * buffers in a fixed 2 MiB array inside the library image, so it calls no
 * cudaMalloc, cudaFree or other allocating routine.
 *   - Same result as nups_push on a store created with deterministic = 1;
 *     NUPS_ESTATE on any other store, or when the store's device is not current.
 *   - n may be at most NUPS_NOALLOC_MAX_ROWS; larger calls return NUPS_EINVAL
 *     (nups_last_cuda_error names the limit) and enqueue nothing.
 *   - The first call on a device looks up the array's device address; make that
 *     first call before any stream capture begins.
 *   - All calls, on all stores of the process, share the one array per device.
 *     It keeps whatever the last call left; every buffer in it is rewritten in
 *     full before it is read, so nothing needs clearing.  Two calls whose work
 *     overlaps on the GPU (different streams, no ordering between them) race on
 *     it: order them, or use nups_push for one of them.                        */
#define NUPS_NOALLOC_MAX_ROWS 65536
nups_status nups_push_noalloc(nups_store* store, const uint32_t* d_keys, uint64_t n, const void* d_delta,
                              void* stream);

/* ---- per-key management (Section 3.2, Section 5.1) ------------------------ */

/* Set the technique of the listed keys.  Pending replica updates are merged
 * first.  NUPS_REPLICATE appends every listed key that is not replicated yet as
 * a new hot slot, in list order (first occurrence); NUPS_SINGLE removes the
 * listed keys and renumbers the remaining slots in their old order.  May
 * allocate; synchronises the stream.                                          */
nups_status nups_set_management(nups_store* store, const uint32_t* d_keys, uint64_t n, int technique, void* stream);

/* sync (Section 3.2: periodic sparse all-reduce of replica updates): for every
 * hot slot touched since the last sync add the workers' pending updates, worker
 * 0 first, to the stored row and clear them (with merge_mean: their sum divided
 * by the number of workers that touched the slot).  With no replicated key
 * nothing is launched.                                                        */
nups_status nups_sync(nups_store* store, void* stream);

/* Add 1 to the access count of every key of the stream (dataset frequency
 * statistics, Section 5.1).                                                   */
nups_status nups_count_accesses(nups_store* store, const uint32_t* d_keys, uint64_t n, void* stream);

/* Copy the num_keys access counts to d_counts_out.                            */
nups_status nups_get_counts(nups_store* store, uint64_t* d_counts_out, void* stream);

/* Choose hot keys from the access counts (Section 5.1).  by_topk = 0: keys with
 * count * num_keys > param * (sum of counts), i.e. more than `param` times the
 * mean (the paper's heuristic uses 100).  by_topk = 1: the `param` most frequent
 * keys.  Output order: count descending, smaller key first among equals.
 * d_keys_out must hold min(param, num_keys) keys for by_topk = 1 and num_keys
 * for the threshold rule; *h_n_out receives the number written.  The largest
 * count and num_keys - 1 must fit 64 bits together (NUPS_ESTATE otherwise).
 * Synchronises the stream.                                                    */
nups_status nups_select_hot(nups_store* store, int by_topk, uint64_t param, uint32_t* d_keys_out, uint64_t* h_n_out,
                            void* stream);

/* Number of replicated keys, and their keys in slot order (d_keys_out may be
 * NULL).  Synchronises the stream when d_keys_out is given.                   */
nups_status nups_get_hot(nups_store* store, uint64_t* h_n_out, uint32_t* d_keys_out, void* stream);

/* Move the listed keys to the worker of their item (the paper's localize,
 * Section 3.1.3); when a key is listed more than once the last item wins.
 * Replicated keys are unaffected.  No-op unless track_ownership.              */
nups_status nups_localize(nups_store* store, const uint32_t* d_keys, uint64_t n, void* stream);

/* Owning worker of each listed key into d_owner_out (int32): the worker, or -2
 * for a replicated key, -1 for a key out of range, -3 if ownership is not
 * tracked.                                                                    */
nups_status nups_get_owner(nups_store* store, const uint32_t* d_keys, uint64_t n, int32_t* d_owner_out, void* stream);

/* ---- sampling access (Sections 4.3, 4.4) ---------------------------------- */

/* register_distribution(pi, level): pi lives on keys [key_base, key_base + n);
 * d_weights[j] is the integer weight of key_base + j, NULL = uniform.  level is
 * one of NUPS_CONFORM .. NUPS_NONCONFORM; U (use frequency) and G (pool size)
 * are used by NUPS_BOUNDED and NUPS_LONGTERM.  Builds the alias table on the
 * device.  Requires n * sum(weights) < 2^64 and G <= 1024.  *h_dist_out receives
 * the distribution id.  Synchronises the stream.                              */
nups_status nups_register_distribution(nups_store* store, uint32_t key_base, const uint32_t* d_weights, uint64_t n,
                                       int level, uint32_t U, uint32_t G, uint64_t seed, int32_t* h_dist_out,
                                       void* stream);

/* Copy a distribution's alias table (thresholds, aliases; n entries each) and
 * return the total weight; for checking a build.                              */
nups_status nups_get_alias_table(nups_store* store, int32_t dist, uint64_t* d_thr_out, uint32_t* d_alias_out,
                                 uint64_t* h_total_weight_out, void* stream);

/* handle = PrepareSample(dist, N): reserve the next N samples.  The N output
 * positions are cut into `workers` contiguous sub-handles; sub-handle q takes
 * the next stretch of worker q's sample stream and (except under NON-CONFORM)
 * localizes its keys to worker q.  Returns without waiting for the device.    */
nups_status nups_prepare_sample(nups_store* store, int32_t dist, uint64_t N, nups_handle* h_out, void* stream);

/* keys, values = PullSample(handle, n): the next n keys of the handle into
 * d_keys_out and, if d_vals_out is not NULL, their rows [n][value_len] as the
 * sub-handle's worker pulls them.  Partial pulls may be of any sizes that add
 * up to N; the handle is released by the pull that completes it.  NUPS_ESTATE
 * when n exceeds what is left.
 *   CONFORM     independent draws from pi.
 *   BOUNDED     pools of G draws, each walked U times in a fresh random order.
 *   LONG-TERM   as BOUNDED, but a sample whose key is not local to the worker
 *               at the start of the call is re-localized and postponed to the
 *               end of its sub-handle, at most once.
 *   NON-CONFORM the first key local to the worker at or after an independent
 *               candidate (64 probes, then the candidate itself).             */
nups_status nups_pull_sample(nups_store* store, nups_handle handle, uint64_t n, uint32_t* d_keys_out,
                             void* d_vals_out, void* stream);

/* ---- workload steps (Section 5.1) ----------------------------------------- */
/* One step over a batch of n items: draw the negatives (one handle of n*K
 * samples from `dist`; item i uses samples i*K .. i*K+K-1), pull, compute, push,
 * localize the item's direct keys to its worker, and merge replicas every
 * sync_interval steps.  deterministic = 1: all pulls see the values from before
 * the step, pushes are applied in item order.  Otherwise items race.
 * d_loss_out (nullable) receives the mean loss over the batch as one float.   */

/* Skip-gram with negative sampling: centre key c, context key o, negatives u_j:
 * x_j = v.u_j, g_j = sigmoid(x_j) - [j = 0], u_j -= lr g_j v, v -= lr sum g_j u_j,
 * loss = -log sigmoid(x_0) - sum_j log sigmoid(-x_j); scores clamped to +-30.
 * K <= 30.                                                                    */
nups_status nups_step_sgns(nups_store* store, const uint32_t* d_center, const uint32_t* d_context, uint64_t n_pairs,
                           int32_t dist, uint32_t K, float lr, float* d_loss_out, void* stream);

/* Many skip-gram steps from one call: n_total pairs are taken as n_total / batch
 * consecutive steps of `batch` pairs, each exactly like one nups_step_sgns
 * (own handle of batch * K negatives, replicas merged every sync_interval
 * steps).  d_loss_out (nullable) receives one mean loss per step.  In fast mode
 * (and without access counting or ownership tracking) the steps between two
 * merges share one kernel launch, so pairs of different steps of that stretch
 * race like pairs of one step do; otherwise the steps run one after the other.
 * A merge that falls due before the call's last step runs on a stream that the
 * library owns, beside the drawing of the next steps' negatives; the next step
 * kernel waits for it, and when the call returns all of its work is ordered on
 * `stream` as usual.  n_total must be a multiple of batch.                     */
nups_status nups_run_sgns(nups_store* store, const uint32_t* d_center, const uint32_t* d_context, uint64_t n_total,
                          uint64_t batch, int32_t dist, uint32_t K, float lr, float* d_loss_out, void* stream);

/* ComplEx with AdaGrad: rows are [re | im]; phi = Re sum h r conj(t); negative j
 * replaces the head when j is even, the tail when odd;
 * loss = softplus(-phi_pos) + sum_j softplus(phi_j); per key role with summed
 * gradient g: acc += g^2, val -= lr g / (sqrt(acc_pulled + g^2) + eps).
 * Needs with_adagrad, value_len <= 512 and K <= 30.                           */
nups_status nups_step_complex(nups_store* store, const uint32_t* d_h, const uint32_t* d_r, const uint32_t* d_t,
                              uint64_t n, int32_t dist, uint32_t K, float lr, float eps, float* d_loss_out,
                              void* stream);

/* Matrix factorization by SGD: e = x - w.h, w += lr (e h - l2 w),
 * h += lr (e w - l2 h), loss = mean e^2.                                      */
nups_status nups_step_mf(nups_store* store, const uint32_t* d_row, const uint32_t* d_col, const float* d_x, uint64_t n,
                         float lr, float l2, float* d_loss_out, void* stream);

/* The same step for cells that arrive column by column (Section 5.1: each worker
 * visits its cells by column, in random order of columns and of the cells within
 * a column, to create locality in the column parameter accesses).  In fast mode
 * a column's row is read once and its updates are summed and added once per
 * stretch of consecutive cells of that column that one warp works on (all cells
 * of such a stretch see the column's row from before the stretch, which is the
 * batch semantics of the deterministic mode).  Any order of cells gives a correct
 * step; the order only decides how much is saved.  In deterministic mode the
 * call is nups_step_mf.  Arguments, ownership and errors as nups_step_mf.      */
nups_status nups_step_mf_by_column(nups_store* store, const uint32_t* d_row, const uint32_t* d_col, const float* d_x,
                                   uint64_t n, float lr, float l2, float* d_loss_out, void* stream);

/* Keys drawn as negatives by the most recent step ([n * K], library-owned
 * device memory, valid until the next step).                                  */
nups_status nups_last_negatives(nups_store* store, const uint32_t** h_d_keys_out, uint64_t* h_n_out);

/* Time-based replica synchronisation (Section 3.2: replicas are synchronised
 * periodically by a background thread and staleness is bounded by time, not by
 * a logical clock; Section 5.6 varies the period from 8 ms to 5 s).  With
 * period_us > 0 a host thread owned by the store enqueues a merge of all
 * replicas every period_us microseconds on a stream of its own, so merging
 * overlaps the caller's work and never blocks it; a tick is skipped while the
 * previous merge is still running.  period_us = 0 stops the ticks and returns
 * once merges already enqueued have finished.  Independent of sync_interval
 * and nups_sync, which keep working (a caller that wants only time-based
 * merging creates the store with sync_interval = 0).
 * Such a merge runs concurrently with pulls, pushes and steps: no update is
 * lost or applied twice, but a pull that overlaps it may miss, for that one
 * read, updates that are just moving from a replica to the stored row.  After
 * nups_set_sync_period(store, 0) and nups_sync every update is in the stored
 * rows.  NUPS_ESTATE on a deterministic store (merges at arbitrary times are not
 * reproducible); nups_create rejects that combination with NUPS_EINVAL.
 * The merge reads every replicated slot of every worker each period: meant for
 * periods of a millisecond and more.                                          */
nups_status nups_set_sync_period(nups_store* store, uint32_t period_us);

/* Gradient-norm clipping for replicated keys (Section 5.1, implementation
 * notes: updates to replicated parameters that exceed the average norm by more
 * than 2x are clipped in the word-vector and matrix-factorization tasks).  With
 * clip_factor > 0 the skip-gram and matrix-factorization steps compare the
 * Euclidean norm of every update row bound for a replicated key with
 * clip_factor times the mean norm of all such updates that earlier steps
 * applied, and scale a longer row down to that bound (direction kept).  The
 * bound is fixed while a step runs (in fast mode: while one launch of
 * nups_run_sgns runs, which may cover several steps); nothing is clipped before
 * the first such update has been applied.  This call returns the statistics:
 * *h_sum = sum of the norms as applied, *h_count = number of updates; it
 * synchronises the stream.                                                    */
nups_status nups_get_clip_stats(nups_store* store, double* h_sum, uint64_t* h_count, void* stream);

/* ---- status and statistics ------------------------------------------------ */

/* Read and clear the device status word (synchronises the stream): NUPS_OK,
 * NUPS_EKEY or NUPS_ETIMEOUT.                                                 */
nups_status nups_status_check(nups_store* store, void* stream);

/* h_out[0..7]: steps, syncs launched, kernels launched by the library so far,
 * accesses served from replicas, accesses served in place, hot slots,
 * background merges enqueued, 0.
 * The two access counters are only kept when count_accesses is set.
 * Synchronises the stream.                                                    */
nups_status nups_get_stats(nups_store* store, uint64_t* h_out, void* stream);

/* Timing aid for benchmarks.  While enabled, the library records a pair of CUDA
 * events on the call's stream around the main kernel of nups_pull*, nups_push*
 * (fast mode) and nups_step_* (the row gather, the scatter-add, the fused step
 * kernel).  nups_kernel_timing only switches the recording on or off (no
 * synchronisation; pairs already recorded stay until they are queried), so a
 * caller can time some repetitions of a loop and leave the others undisturbed:
 * an event between two kernels keeps the second from starting while the first
 * drains.  nups_kernel_time synchronises the stream, adds up the elapsed
 * times of all pairs recorded since the last query, returns the sum in
 * milliseconds and the number of launches, and starts afresh.                 */
nups_status nups_kernel_timing(nups_store* store, int enable);
nups_status nups_kernel_time(nups_store* store, double* h_ms_out, uint64_t* h_launches_out, void* stream);

/* The same, kept apart by kind of kernel: h_ms_out[8] and h_launches_out[8] receive, at index
 * 0 the row gather of nups_pull*, 1 the scatter-add of nups_push* (fast mode), 2 the fused kernel of
 * nups_step_*, 3 the row copy of nups_pull_sample, 4 the draw kernel of nups_prepare_sample; the
 * other entries are zero.  Synchronises the stream and starts afresh, like nups_kernel_time.     */
nups_status nups_kernel_times(nups_store* store, double* h_ms_out, uint64_t* h_launches_out, void* stream);

/* Measurement aid: the rate at which this GPU applies 128-bit floating-point
 * reductions (red.global.add.v4.f32, the instruction every fast-mode update
 * uses) to distinct, streaming addresses.  Adds zeros to the first `bytes` bytes
 * of the value table `reps` times (the table is unchanged) and returns the
 * payload rate in GB/s.  This is the ceiling of push and of the workload steps
 * in fast mode.  Synchronises the stream.                                      */
nups_status nups_probe_reduction_rate(nups_store* store, uint64_t bytes, uint32_t reps, double* h_gbs_out, void* stream);

/* ---------------------------------------------------------------------------
 * A value table partitioned over several GPUs (Section 3.1: the servers of a
 * parameter server hold disjoint parts of the parameters, classically by key
 * range; Section 3.2: a worker reaches a parameter held elsewhere through that
 * node).  Among GPUs of one NVLink domain the owner's memory is addressable, so
 * the access is made by the calling GPU's own kernel: pull loads the row from
 * the owner's memory, push adds to it there with floating-point reductions.
 * No message, no exchange of keys, no work on the owner.
 *
 * Shard j holds the fp32 rows of keys [j * kps, (j + 1) * kps), kps =
 * ceil(num_keys / n_shards).  Every process creates one object for its own
 * shard (my_shard), which allocates and zero-fills that shard on the current
 * device, and attaches the first-row address of every other shard:
 *   - a pointer valid in this process (a shard of another object of the same
 *     process; for another device the caller has enabled peer access), or
 *   - the handle another process exported for its shard (CUDA IPC; peer access
 *     is enabled by the mapping).
 * Handles are plain bytes: ship them with whatever the processes use to talk
 * (torch.distributed, a file).  An attached shard must outlive the attachment.
 * Values are fp32; keys out of range are skipped as in the store (a pulled row
 * is zero-filled, nups_shard_status_check reports NUPS_EKEY).  Not replicated:
 * keys hot enough to be replicated belong in a per-GPU nups_store.
 * Ordering: calls are stream-ordered on the calling GPU only.  Updates pushed
 * by another GPU are seen by a pull that is ordered after them by the caller's
 * own means (an event, a barrier between processes); additions to one row from
 * several GPUs at once all arrive, in no defined order.
 * nups_shard_pull / nups_shard_push return NUPS_ESTATE until every shard is
 * attached.  Errors of the CUDA runtime: NUPS_ECUDA, text from
 * nups_shard_last_error.                                                      */
typedef struct nups_shard_table nups_shard_table;
#define NUPS_MAX_SHARDS 16
#define NUPS_SHARD_HANDLE_BYTES 64
nups_status nups_shard_table_create(uint64_t num_keys, uint32_t value_len, uint32_t n_shards, uint32_t my_shard,
                                    nups_shard_table** out);
void nups_shard_table_destroy(nups_shard_table* table);
/* device address and size in bytes of this process's shard (for same-process attachment and for filling it) */
nups_status nups_shard_table_local(nups_shard_table* table, void** h_ptr_out, uint64_t* h_bytes_out);
/* whole-shard copy between the local shard and a device buffer of kps * value_len floats (to_table != 0: into the shard) */
nups_status nups_shard_table_copy(nups_shard_table* table, void* d_rows, int to_table, void* stream);
/* handle of the local shard for another process: NUPS_SHARD_HANDLE_BYTES bytes written to h_handle_out */
nups_status nups_shard_table_export(nups_shard_table* table, unsigned char* h_handle_out);
nups_status nups_shard_table_attach(nups_shard_table* table, uint32_t shard, void* d_first_row);
nups_status nups_shard_table_attach_ipc(nups_shard_table* table, uint32_t shard, const unsigned char* h_handle);
/* d_out / d_delta: [n][value_len] fp32, 16-byte aligned, on the calling GPU */
nups_status nups_shard_pull(nups_shard_table* table, const uint32_t* d_keys, uint64_t n, void* d_out, void* stream);
nups_status nups_shard_push(nups_shard_table* table, const uint32_t* d_keys, uint64_t n, const void* d_delta, void* stream);
/* synchronises the stream; NUPS_EKEY once after a key out of range was seen */
nups_status nups_shard_status_check(nups_shard_table* table, void* stream);
const char* nups_shard_last_error(const nups_shard_table* table);

/* Merging a whole store across GPUs (Section 3.2: replicas are synchronised by
 * an all-reduce of the updates they have accumulated).  Use: every GPU holds a
 * nups_store of the same keys (the keys replicated across GPUs: a small store)
 * and pulls and pushes it on its own.  `which` = 0 value table, 1 accumulator.
 *   nups_merge_mark    all GPUs hold the same table now (after the same
 *                      initialisation): remember it as the agreed state.
 *                      Allocates num_keys rows (NUPS_ENOMEM under the limit).
 *   nups_merge_export  merges the store's own replicas (nups_sync), then writes
 *                      own = table - agreed into d_own_out ([num_keys][value_len],
 *                      the store's value type).  NUPS_ESTATE before a mark.
 *   (the caller sums the exported buffers over all GPUs into d_total: one
 *    all-reduce with NCCL or any other transport; d_own must keep its content)
 *   nups_merge_apply   table += d_total - d_own (by reductions, so pushes may
 *                      run beside it), agreed += d_total.
 * Afterwards every GPU's table is the agreed state plus what that GPU added
 * since its export; nothing pushed between export and apply is lost.  With one
 * GPU (d_total = d_own) the table is unchanged.                               */
nups_status nups_merge_mark(nups_store* store, int which, void* stream);
nups_status nups_merge_export(nups_store* store, int which, void* d_own_out, void* stream);
nups_status nups_merge_apply(nups_store* store, int which, const void* d_total, const void* d_own, void* stream);

const char* nups_strerror(nups_status status);
const char* nups_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* NUPS_H */
