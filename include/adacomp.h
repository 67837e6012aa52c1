/*
 * libadacomp: the data-parallel hot path of AdaComp (Hardy, Le Merrer, Sericola,
 * "Distributed deep learning on edge-devices: feasibility via adaptive
 * compression") for NVIDIA B200 (sm_100a).
 *
 *   worker side   SELECT_GRAD (Algorithm 1): per tensor V_l / beta_l keep the
 *                 k_l entries of largest magnitude and emit them as ascending
 *                 (index, value) pairs;
 *   server side   the body of Algorithm 2: for every entry of an arriving update
 *                 compute the per-parameter staleness sigma_k (Eq. 3), the
 *                 learning rate alpha_k (Eq. 5) and the new Theta_k (Eq. 4), and
 *                 advance the timestamp once per update.
 *
 * Conventions that hold for every entry point
 *   - Plain C ABI.  Every call returns an adacomp status (0 = ADACOMP_OK, negative
 *     = error); nothing throws, aborts or exits.
 *   - Pointers named d_* are DEVICE pointers, pointers named h_* are HOST pointers.
 *     All device memory is owned by the caller.  The library never allocates
 *     device memory: handles carve their scratch out of the caller's workspace
 *     (size from the *_workspace_bytes calls, base aligned to 256 bytes), which
 *     must stay valid until the handle is destroyed.  Handles themselves are small host
 *     allocations of the library.
 *   - cuda_stream is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Device work is enqueued on it and the call returns without
 *     waiting.  Argument errors are returned at once, before anything is
 *     enqueued; errors that only the device can see are returned by the
 *     *_last_error calls, which wait for the stream.
 *   - A handle belongs to one device and is not thread-safe; use it from one
 *     stream at a time.
 */
#ifndef ADACOMP_H_
#define ADACOMP_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define ADACOMP_API __attribute__((visibility("default")))
#else
#define ADACOMP_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

enum {
    ADACOMP_OK = 0,
    ADACOMP_ERR_INVALID = -1,       /* null pointer, k > n, bad size, misaligned workspace ...   */
    ADACOMP_ERR_ALLOC = -2,         /* host allocation failed, or workspace too small           */
    ADACOMP_ERR_CUDA = -3,          /* a CUDA runtime call failed (see adacomp_last_cuda_error)  */
    ADACOMP_ERR_WINDOW = -4,        /* pull timestamp j > i, or j older than the kept history   */
    ADACOMP_ERR_CAPACITY = -5,      /* more pairs / updates than the server was created for     */
    ADACOMP_ERR_UNSORTED = -6,      /* an update's indices are not strictly ascending / in range */
    ADACOMP_ERR_TIMEOUT = -7,       /* reserved: a bounded device-side wait gave up             */
    ADACOMP_ERR_UNIMPLEMENTED = -8
};

/* Static text for a status code ("ok", "invalid argument", ...). Never NULL. */
ADACOMP_API const char* adacomp_status_string(int status);
/* Library version, major * 10000 + minor * 100 + patch. */
ADACOMP_API int adacomp_version(void);
/* The last cudaError_t (as int) a call of this library saw on the calling thread, 0 if none. */
ADACOMP_API int adacomp_last_cuda_error(void);
/* How many kernels this library has launched in this process so far (all handles, all threads). */
ADACOMP_API uint64_t adacomp_kernel_launches(void);

/* ------------------------------------------------------------------------------------------
 * Worker side: SELECT_GRAD (Algorithm 1; "Selection method" paragraph).
 * ---------------------------------------------------------------------------------------- */

/* One selection unit: a tensor V_l or beta_l occupying entries [offset, offset + n) of the
 * worker's gradient vector, of which the k entries of largest |value| are kept.  Segments
 * must not overlap and must be listed by ascending offset. */
typedef struct {
    uint64_t offset;
    uint32_t n;
    uint32_t k;
} adacomp_segment_t;

/* k for a keep fraction c = c_num / c_den ("the (100 x c)% largest", Algorithm 1):
 * k = min(n, max(1, ceil(n * c_num / c_den))) in exact integer arithmetic; n = 0 gives 0.
 * The paper does not state the rounding; the ceiling keeps every tensor represented.
 * ADACOMP_ERR_INVALID on c_den = 0, c_num > c_den, n >= 2^32 or k_out = NULL. */
ADACOMP_API int adacomp_keep_count(uint64_t n, uint32_t c_num, uint32_t c_den, uint32_t* k_out);

typedef struct adacomp_select adacomp_select_t;

/* Bytes of device workspace adacomp_select_create needs for this layout and up to max_workers
 * gradient vectors per call.  ADACOMP_ERR_INVALID on a bad layout (k > n, overlap, unsorted,
 * total entries or pairs beyond 2^32 - 2, n_segs = 0, max_workers = 0). */
ADACOMP_API int adacomp_select_workspace_bytes(const adacomp_segment_t* h_segs, uint32_t n_segs,
                                   uint32_t max_workers, size_t* bytes_out);

/* Creates a selector for a fixed layout on CUDA device `device`.  The paper keeps no state on
 * the worker between iterations (Algorithm 1 pulls, computes, selects, pushes), so neither
 * does the handle: it only holds the layout and scratch.  d_workspace: device memory,
 * 256-byte aligned, at least the size reported above.  Synchronous (copies the layout to the
 * device and clears scratch).  On error *h is NULL. */
ADACOMP_API int adacomp_select_create(adacomp_select_t** h, const adacomp_segment_t* h_segs, uint32_t n_segs,
                          uint32_t max_workers, void* d_workspace, size_t workspace_bytes, int device);

/* SELECT_GRAD for n_workers gradient vectors at once.
 *   d_grads              fp32, worker w's vector starts at d_grads + w * worker_stride_elems;
 *                        4-byte aligned; read only, never modified; NaN-free by contract
 *                        (a NaN orders above +Inf by bit pattern, deterministically).
 *   d_idx_out, d_val_out [n_workers][K] with K = sum of k over the segments: worker w's pairs
 *                        start at w * K, segment after segment, ascending index inside a
 *                        segment.  idx is the position in the gradient vector (offset + e);
 *                        val is the gradient entry itself, bit for bit.  Fully overwritten.
 * Selection rule: order entries of a segment by (bits & 0x7FFFFFFF) descending, then by index
 * ascending, and keep the first k: equal magnitudes are resolved in favour of the lower index,
 * +0 and -0 tie.  Entries not kept are dropped; no residual is accumulated.
 * Errors: ADACOMP_ERR_INVALID (null pointer, n_workers = 0 or > max_workers,
 * worker_stride_elems smaller than the layout's extent), ADACOMP_ERR_CUDA. */
ADACOMP_API int adacomp_select(adacomp_select_t* h, const float* d_grads, uint64_t worker_stride_elems,
                   uint32_t n_workers, uint32_t* d_idx_out, float* d_val_out, void* cuda_stream);

/* Same operation for callers whose gradients live in host memory: copies h_grads to the
 * caller's device staging buffers, selects, and copies the pairs back.  h_* buffers should be
 * pinned for the copies to be asynchronous; they must stay untouched until the stream has
 * drained.  d_grads_staging holds n_workers * worker_stride_elems floats; d_idx_staging and
 * d_val_staging hold n_workers * K entries each. */
ADACOMP_API int adacomp_select_host(adacomp_select_t* h, const float* h_grads, uint64_t worker_stride_elems,
                        uint32_t n_workers, float* d_grads_staging, uint32_t* d_idx_staging,
                        float* d_val_staging, uint32_t* h_idx_out, float* h_val_out,
                        void* cuda_stream);

/* Chooses how selections are computed; the results are identical.
 * 0 = automatic: tensors of at least 32768 entries with k <= n/4 take the bracketed route (a
 *     sample brackets the threshold, then the gradient is read once); shorter tensors are
 *     selected whole in shared memory (read once); instances whose bracket turns out wrong (or
 *     that hold a NaN), and longer tensors with k > n/4, take the general route;
 * 1 = general route for everything (multi-pass radix select; reads the gradient five times);
 * 2 = as 0, but tensors of a million entries or more whose candidates fit take the cluster route: one
 *     thread-block cluster per (worker, tensor) keeps masks and candidate values in its distributed
 *     shared memory between the single pass and the ordered write, so DRAM sees the gradient once and
 *     the output once and nothing else.  Measured slower than 0 on a B200 (its blocks can hold fewer
 *     warps, and a cluster's steps run one after the other), hence not the default. */
ADACOMP_API int adacomp_select_set_route(adacomp_select_t* h, int route);

/* How the handle's layout is mapped on this device: h_info_out[0] = tensors on the cluster route (large
 * tensors selected by one thread-block cluster each, everything between the one pass over the gradient and
 * the ordered write kept in the cluster's shared memory), [1] = blocks per cluster, [2] = buffers per warp
 * in its ring of bulk copies + 256 x warps per block, [3] = clusters the device keeps resident.  All 0 if
 * no tensor is on that route. */
ADACOMP_API int adacomp_select_route_info(const adacomp_select_t* h, uint32_t* h_info_out);

/* Stage timing.  With profiling on (on = 1), every adacomp_select call records CUDA events on its stream
 * around each of its kernels (no synchronisation; the events between the kernels cost some ten
 * microseconds per call on the device); on = 2 records them around the one pass over the gradient
 * only (stage "bracket_scan"), which leaves the call's own duration practically untouched.
 * adacomp_select_profile waits for the calls made since profiling was switched on and writes
 * the mean device time per call of each stage, in milliseconds, to h_ms_out[0 .. n_stages),
 * n_stages = the number of stages adacomp_select_stage_name knows (0 for a stage that never ran),
 * and the number of calls to *h_calls_out (may be NULL).  Switching profiling on (again) starts a fresh measurement.
 * adacomp_select_stage_name names a stage ("bracket_scan", ...; "" beyond the last). */
ADACOMP_API int adacomp_select_set_profiling(adacomp_select_t* h, int on);
ADACOMP_API int adacomp_select_profile(adacomp_select_t* h, float* h_ms_out, uint32_t n_stages,
                                       uint64_t* h_calls_out);
ADACOMP_API const char* adacomp_select_stage_name(uint32_t stage);

/* K = sum of k over the layout's segments (pairs per worker). */
ADACOMP_API int adacomp_select_pairs_per_worker(const adacomp_select_t* h, uint64_t* pairs_out);
/* Values of entries chosen elsewhere: d_val_out[w][e] = d_grads[w][d_idx[w][e]] for the handle's
 * K = pairs_per_worker entries of each of n_workers workers (same layouts as adacomp_select).
 * Serves selections the library does not make itself, e.g. the random subset that one variant
 * of Comp-ASGD sends instead of the largest entries ("Compression" paragraph); the random draw
 * is the caller's.  An index outside the layout's extent
 * reads as 0 and is reported by adacomp_select_last_error as ADACOMP_ERR_INVALID. */
ADACOMP_API int adacomp_select_gather(adacomp_select_t* h, const float* d_grads, uint64_t worker_stride_elems,
                                      uint32_t n_workers, const uint32_t* d_idx, float* d_val_out,
                                      void* cuda_stream);

/* Waits for cuda_stream, then returns the first error the device recorded since the last call
 * of this function (ADACOMP_OK if none) and clears it.  Also reports, if stats_out is not
 * NULL, stats_out[0] = how many (worker, segment) selections of the last adacomp_select call
 * took the general multi-pass route rather than one of the two single-pass routes. */
ADACOMP_API int adacomp_select_last_error(adacomp_select_t* h, void* cuda_stream, uint64_t* stats_out);
ADACOMP_API int adacomp_select_destroy(adacomp_select_t* h);

/* Selection of ONE tensor for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a convenience of this library.)  Same rule and same output as
 * adacomp_select for a single segment {offset 0, n, k} and a single worker: the k entries of
 * largest magnitude of d_grad[0 .. n), lower index first among equals, written by ascending
 * index to d_idx_out[0 .. k) / d_val_out[0 .. k).  No handle and no workspace: the scratch the
 * selection needs (11 008 bytes) is a fixed array inside the library, present on every GPU that
 * loads it for as long as the process lives; the call allocates nothing, on the host or on the
 * device, and frees nothing.  Meant for code that runs where an allocation is not an option:
 * inside another framework's step whose memory pool it cannot reach, in a loop whose memory was
 * budgeted at start-up, or while an allocation would stall or fail.
 *   n <= 16 777 216 (2^24) entries; a larger n is refused with ADACOMP_ERR_CAPACITY and nothing
 *   is enqueued.  k <= n; k = 0 does nothing.  d_grad must be 4-byte aligned.
 *   The first call on a device looks up the array's device address (a CUDA runtime query, done
 *   once per device with that device current); make that first call before any stream capture.
 *   All calls on a device share the one array, which keeps whatever the previous call left
 *   (every call clears what it needs zeroed): two calls whose device work overlaps, on two
 *   streams or from two threads, race on it.  Keep calls on a device in one stream, or order
 *   them with events.
 * Work is enqueued on cuda_stream; the call returns without waiting. */
ADACOMP_API int adacomp_select_static(const float* d_grad, uint32_t n, uint32_t k, uint32_t* d_idx_out,
                                      float* d_val_out, int device, void* cuda_stream);
/* Companion of adacomp_select_static (no counterpart in the paper either): waits for cuda_stream,
 * then returns the first error the device recorded during adacomp_select_static calls on `device`
 * since the last call of this function (ADACOMP_OK if none) and clears it.  The status word is
 * part of the same built-in array: nothing is allocated and the caller passes no buffer. */
ADACOMP_API int adacomp_select_static_last_error(int device, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Server side: Algorithm 2 (Eq. 3, Eq. 4, Eq. 5; "Complexity" paragraph for the history).
 * ---------------------------------------------------------------------------------------- */

typedef struct adacomp_server adacomp_server_t;

/* Bytes of device workspace for a server over n_params parameters that remembers the last
 * history_pairs (index, value) pairs it applied.  The paper's server keeps the index lists of
 * the last d updates (d = worst delay, of the order of the number of workers); here the bound
 * is expressed in pairs: an update whose pull timestamp j is so old that update j's pairs have
 * been overwritten is refused with ADACOMP_ERR_WINDOW. */
ADACOMP_API int adacomp_server_workspace_bytes(uint64_t n_params, uint64_t history_pairs, size_t* bytes_out);

/* Creates the server state on `device`: timestamp, per-parameter history heads and the ring of
 * the last history_pairs pairs.  max_window_updates bounds i - j for any update (and how many
 * updates one adacomp_apply call may carry); it must be < 2^24 so that sigma converts to fp32
 * exactly.  n_params <= 2^32 - 2, history_pairs < 2^31.  Synchronous.  The server is unusable
 * until adacomp_server_reset has given it a parameter vector. */
ADACOMP_API int adacomp_server_create(adacomp_server_t** s, uint64_t n_params, uint64_t history_pairs,
                          uint32_t max_window_updates, void* d_workspace, size_t workspace_bytes,
                          int device);

/* First step of Algorithm 2 (the initial parameters): adopts d_theta (n_params fp32, caller-owned, holding
 * the initial values) as the parameter vector that adacomp_apply updates in place, sets the
 * timestamp to 0 and forgets all history.  The buffer must outlive the server or the next
 * reset. */
ADACOMP_API int adacomp_server_reset(adacomp_server_t* s, float* d_theta, void* cuda_stream);

/* Pull_Theta (Algorithm 1): reports the current timestamp i in *h_timestamp_out and, if
 * d_theta_copy is not NULL, enqueues a copy of the n_params parameters into it. */
ADACOMP_API int adacomp_server_pull(adacomp_server_t* s, float* d_theta_copy, uint64_t* h_timestamp_out,
                        void* cuda_stream);

/* Get + loop body of Algorithm 2 for n_updates arriving updates, strictly in array order
 * (= arrival order).  Update b consists of the h_pair_count[b] pairs that start at pair
 * h_pair_begin[b] of d_idx / d_val (updates may sit anywhere in those arrays, e.g. worker by
 * worker as adacomp_select wrote them, while arrival order is a permutation of the workers)
 * and of the timestamp h_pull_ts[b] that its worker received with its pull (Push(update, j)).
 * With i the server timestamp when update b is applied, for each of its pairs (k, v):
 *     sigma_k = number of updates u in [j, i-1] that changed Theta_k with a non-zero value (Eq. 3)
 *     alpha_k = lr / sigma_k if sigma_k != 0 else lr                                     (Eq. 5)
 *     Theta_k = Theta_k - alpha_k * v                                                    (Eq. 4)
 * in fp32 with one IEEE rounding per operation (true division, multiply, subtract; no fused
 * multiply-add), then i advances by one (also for an update with no pairs).  A pair whose value
 * is +-0 is not a change (Eq. 3 tests the value): it leaves Theta_k untouched and is not
 * counted by later updates; its sigma is still reported.  Parameters not named by an update are
 * not touched.  Since each parameter sees its updates in arrival order, Theta is bit-identical
 * to one-at-a-time application.
 *   d_idx          indices into Theta, strictly ascending inside one update (what
 *                  adacomp_select emits); d_val the matching values.
 *   h_pair_begin, h_pair_count, h_pull_ts   [n_updates] host arrays.
 *   d_sigma_out    NULL, or device array addressed like d_idx that receives sigma_k per pair.
 * Host-side checks happen before anything is enqueued and leave the server unchanged:
 * ADACOMP_ERR_WINDOW (j > i, i - j > max_window_updates, or update j's pairs already evicted
 * from the history ring), ADACOMP_ERR_CAPACITY (n_updates > max_window_updates, or one call's
 * pairs exceed history_pairs), ADACOMP_ERR_INVALID.  On the device an index >= n_params is
 * skipped and reported by adacomp_server_last_error as ADACOMP_ERR_UNSORTED; with validation
 * switched on (adacomp_server_set_validation) so is an index that is not larger than its
 * predecessor in the same update.  ADACOMP_ERR_ALLOC: a host-side table could not be allocated
 * (nothing enqueued, server unchanged).  If a kernel launch itself fails (ADACOMP_ERR_CUDA) after
 * earlier launches of the same call were enqueued, the device's history is ahead of the host's
 * bookkeeping: the server then refuses every further update with ADACOMP_ERR_CUDA until
 * adacomp_server_reset. */
ADACOMP_API int adacomp_apply(adacomp_server_t* s, const uint32_t* d_idx, const float* d_val,
                              const uint64_t* h_pair_begin, const uint32_t* h_pair_count,
                              const uint64_t* h_pull_ts, uint32_t n_updates, float lr,
                              uint32_t* d_sigma_out, void* cuda_stream);

/* Same operation for updates that arrive in host memory (the server's ingress): copies the
 * range of pairs the updates span from h_idx / h_val into the caller's device staging buffers
 * (same addressing) and applies them.  h_sigma_out may be NULL; if not, it receives sigma per
 * pair through d_sigma_staging, which must then be given too. */
ADACOMP_API int adacomp_apply_host(adacomp_server_t* s, const uint32_t* h_idx, const float* h_val,
                                   const uint64_t* h_pair_begin, const uint32_t* h_pair_count,
                                   const uint64_t* h_pull_ts, uint32_t n_updates, float lr,
                                   uint32_t* d_idx_staging, float* d_val_staging,
                                   uint32_t* d_sigma_staging, uint32_t* h_sigma_out, void* cuda_stream);

/* Current timestamp i = number of updates applied since the last reset (host-side counter). */
ADACOMP_API int adacomp_server_timestamp(const adacomp_server_t* s, uint64_t* h_timestamp_out);
/* on != 0: every apply also checks on the device that indices are in range and strictly
 * ascending inside an update.  Off by default. */
ADACOMP_API int adacomp_server_set_validation(adacomp_server_t* s, int on);
/* Chooses how adacomp_apply maps work to the GPU; results are identical.
 * 0 = automatic: per launch of up to 32 updates, 3 when the launch's pairs number 8 % of the
 *     parameters or more, else 2; a single update goes as 1;
 * 1 = one launch per update, one thread per pair;
 * 2 = up to 32 updates per launch; a warp owns a run of parameter ranges, lines up all pairs of
 *     a range in arrival order and applies them 32 at a time straight on global memory (lanes
 *     that hold the same parameter take turns); only the named parameters are touched;
 * 3 = up to 32 updates per launch over a dense sweep: a warp owns a run of ranges of 128 to 512
 *     parameters (sized to the updates' density), brings Theta and the history heads of a range
 *     into shared memory whole, applies the updates' pairs of the range there (thin updates: all
 *     lined up in arrival order, 32 at a time; dense updates: one update after the other) and
 *     writes back what changed (needs Theta on a 16-byte boundary, else 2 is used).
 * 4 = the paper's own history structure ("Complexity" paragraph) instead of the chains: the ring
 *     keeps the sorted index lists of the recent updates and sigma_k is found with one dichotomous
 *     search per update of the window; one launch per update.  Windows are bounded to 448 updates
 *     (ADACOMP_ERR_WINDOW beyond).  Same results; O((i - j) log K) probes per pair.  Because the
 *     ring then holds another kind of history, mode 4 can only be entered or left while the
 *     timestamp is 0 (ADACOMP_ERR_INVALID otherwise).
 * Updates whose pair slices overlap in memory, with d_sigma_out given, always go as 1: their
 * staleness slots are shared and the later update's count must be the one that stays. */
ADACOMP_API int adacomp_server_set_mode(adacomp_server_t* s, int mode);
/* Which rule adacomp_apply follows.
 * 0 = AdaComp (default): per-parameter staleness sigma_k of Eq. 3, learning rate of Eq. 5.
 * 1 = the competitors' rule of the "Experimental setup" (ASGD, Comp-ASGD: one learning rate per
 *     update, the base rate over the update's staleness): every entry of an update that pulled
 *     at j and is applied at timestamp i gets alpha / (i - j) (alpha if i = j), Eq. 4 is applied
 *     to every entry as written (zero-valued ones too), d_sigma_out receives i - j, and no history
 *     is read or kept.  ADACOMP_ERR_WINDOW if j > i or i - j >= 2^24.
 * The rule can only be changed while the timestamp is 0 (after create or reset): ADACOMP_ERR_INVALID
 * otherwise. */
ADACOMP_API int adacomp_server_set_rule(adacomp_server_t* s, int rule);
/* A dense update under rule 1 (ASGD pushes the whole gradient): Theta <- Theta - alpha / (i - j) *
 * d_delta, d_delta[n_params] in device memory; the timestamp advances by one.
 * ADACOMP_ERR_INVALID under rule 0 (a dense AdaComp update is adacomp_apply with every index). */
ADACOMP_API int adacomp_apply_dense(adacomp_server_t* s, const float* d_delta, uint64_t pull_ts, float lr,
                                    void* cuda_stream);
/* Test hook: advances the history position counter as if `count` more pairs had been applied
 * (their history is empty).  Lets a test reach the 32-bit position re-basing that otherwise
 * happens once per ~4 * 10^9 applied pairs.  Call right after adacomp_server_reset. */
ADACOMP_API int adacomp_server_debug_skip_positions(adacomp_server_t* s, uint64_t count);
/* Waits for cuda_stream, returns and clears the first error recorded on the device. */
ADACOMP_API int adacomp_server_last_error(adacomp_server_t* s, void* cuda_stream);
ADACOMP_API int adacomp_server_destroy(adacomp_server_t* s);

/* ---- index coding -------------------------------------------------------------------------
 * The paper leaves the encoding of the pairs open (footnote of "Algorithm details"); this is a
 * lossless coding of the index half (values travel as they are).  A worker's index list of
 * pairs_per_worker entries, ascending as adacomp_select emits it, is cut into blocks of 256
 * entries; a block is stored as: the first index; w = the number of bits of the largest gap in
 * the block (gap of an entry = index - previous index - 1, modulo 2^32, so any list survives the
 * round trip); the gaps of the block's other entries, w bits each, entry e at bit (e - 1) * w
 * of a little-endian bit string held in 32-bit words.  d_block_off[w][b] (n_blocks + 1 entries
 * per worker, n_blocks = ceil(pairs_per_worker / 256)) is the word at which block b starts in
 * worker w's stream d_words + w * words_per_worker; the last entry is the stream's length.
 * words_per_worker must be at least adacomp_encode_capacity_words(pairs_per_worker)
 * (ADACOMP_ERR_CAPACITY otherwise).  All arrays are the caller's device memory.  Decoding does not
 * trust the stream: a block whose offset, width (> 32) or payload would reach outside the worker's
 * words_per_worker words is not read; all its entries decode to 0xFFFFFFFF, an index that
 * adacomp_apply skips and reports (ADACOMP_ERR_UNSORTED). */
ADACOMP_API uint64_t adacomp_encode_capacity_words(uint64_t pairs_per_worker);
ADACOMP_API int adacomp_encode_indices(const uint32_t* d_idx, uint64_t pairs_per_worker, uint32_t n_workers,
                                       uint32_t* d_words, uint64_t words_per_worker, uint64_t* d_block_off,
                                       int device, void* cuda_stream);
ADACOMP_API int adacomp_decode_indices(const uint32_t* d_words, uint64_t words_per_worker,
                                       const uint64_t* d_block_off, uint64_t pairs_per_worker,
                                       uint32_t n_workers, uint32_t* d_idx_out, int device, void* cuda_stream);

/* ---- value packing ------------------------------------------------------------------------
 * The value half of the same open point (footnote of "Algorithm details"), lossless: every fp32
 * bit pattern comes back as it went in, so Eq. 4 sees the same inputs.  A worker's
 * pairs_per_worker values are cut into blocks of 256 entries, like the indices.  With E(x) the
 * 8-bit exponent field of x, a block is stored as: one word e_min | w_e << 8 (e_min the smallest
 * E in the block, w_e the number of bits of the largest E - e_min, 0 .. 8); then the block's n
 * entries, 24 + w_e bits each, entry t at bit t * (24 + w_e) of a little-endian bit string held in
 * 32-bit words, an entry being the 23 mantissa bits, above them E - e_min in w_e bits, above
 * that the sign.  (The largest magnitudes of a tensor lie within a few powers of two of each
 * other: 26 or 27 bits a value.)  d_block_off and d_words are laid out as for the indices;
 * words_per_worker must be at least adacomp_encode_values_capacity_words(pairs_per_worker)
 * (ADACOMP_ERR_CAPACITY otherwise).  All arrays are the caller's device memory.  Decoding does not
 * trust the stream: a block whose header has w_e > 8 or other bits set, or whose offset or
 * payload would reach outside the worker's words_per_worker words, is not read; all its entries
 * decode to +0.0, a value that changes no parameter, and so does an entry whose exponent would
 * come out above 255. */
ADACOMP_API uint64_t adacomp_encode_values_capacity_words(uint64_t pairs_per_worker);
ADACOMP_API int adacomp_encode_values(const float* d_val, uint64_t pairs_per_worker, uint32_t n_workers,
                                      uint32_t* d_words, uint64_t words_per_worker, uint64_t* d_block_off,
                                      int device, void* cuda_stream);
ADACOMP_API int adacomp_decode_values(const uint32_t* d_words, uint64_t words_per_worker,
                                      const uint64_t* d_block_off, uint64_t pairs_per_worker,
                                      uint32_t n_workers, float* d_val_out, int device, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* ADACOMP_H_ */
