/*
 * dgc.h -- C ABI of the B200-native Deep Gradient Compression hot path.
 *
 * One `dgc_state` is one worker ("node k" of Algorithm 4, Appendix D): it owns
 * the two accumulators U^k and V^k of that algorithm for a whole gradient set
 * (tensors j = 0..M laid out in one fp32 arena) and compresses one gradient
 * per call.  The receive side (`dgc_decode_accumulate`, `dgc_apply_sgd`) is
 * stateless.
 *
 * Conventions
 *  - "device" pointers are CUDA device memory of the state's device, owned by
 *    the caller unless stated; "host" pointers are ordinary host memory.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *    Calls that take a stream only enqueue work on it and return without
 *    synchronising, unless stated.
 *  - Every function returns DGC_OK (0) or a negative DGC_E* code; nothing
 *    throws, aborts or prints.  dgc_error_string() names a code.
 *  - There is no CPU fallback: without a usable CUDA device every call that
 *    needs one returns DGC_ECUDA.
 *
 * Arena layout: tensor j occupies arena[arena_offset[j] .. + numel[j]); every
 * tensor starts on a multiple of DGC_ARENA_ALIGN elements and the arena length
 * is a multiple of it (dgc_layout reports the offsets).  The slots between
 * tensors are padding: never selected, never written in u/v, decoded as +0.
 * Their content in the gradient arena is ignored (it may be anything).
 */
#ifndef DGC_H_
#define DGC_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DGC_OK          0
#define DGC_EINVAL     -1   /* bad argument                                   */
#define DGC_ENOMEM     -2   /* device or host allocation failed               */
#define DGC_ECAPACITY  -3   /* output buffer smaller than dgc_max_nnz()       */
#define DGC_ECUDA      -4   /* a CUDA runtime call or kernel launch failed    */
#define DGC_ESTATE     -5   /* state handle is NULL or already destroyed      */

#define DGC_ARENA_ALIGN        512   /* elements; tensor starts and arena length */
#define DGC_MAX_DECODE_WORKERS 64
#define DGC_STATIC_DECODE_WORDS (1 << 18)   /* int32 words of built-in decode scratch (1 MiB) */

/* dgc_status.flags */
#define DGC_FLAG_NONFINITE_NORM   1  /* the clipping norm was Inf or NaN            */
#define DGC_FLAG_FULL_SELECT      2  /* a tensor needed the full-tensor selection   */
#define DGC_FLAG_CAND_OVERFLOW    4  /* sampled threshold let too many entries pass */
#define DGC_FLAG_CAND_SHORT       8  /* sampled threshold let fewer than k pass     */
#define DGC_FLAG_TIE_FILL        16  /* fewer than k entries of a tensor exceeded   */
                                     /* the sample's key: entries tied with it (all */
                                     /* zeros, few distinct magnitudes) complete    */
                                     /* the list, lowest indices first; not slow    */

typedef struct dgc_state dgc_state;   /* opaque */

typedef struct dgc_config {
  int32_t        num_tensors;     /* M+1 of Algorithm 4; >= 1                                   */
  int32_t        num_workers;     /* N: only enters the clip threshold thr_G * N^-1/2 (App. C)  */
  const int64_t* tensor_numel;    /* host array [num_tensors], each >= 1; copied                */
  float          momentum;        /* m of Eq. 5                                                 */
  float          clip_threshold;  /* thr_G of Appendix C before the N^-1/2 scaling; <= 0: off   */
  double         sparsity;        /* s in [0, 1): fraction of each tensor that is NOT sent      */
  double         sample_ratio;    /* fraction of |v| sampled for the threshold estimate
                                     (Sec. 5: 0.1% .. 1%); 0 selects the default 0.01           */
  uint64_t       seed;            /* seed of the sampling positions                             */
  int32_t        device;          /* CUDA device ordinal                                        */
  int32_t        debug_sample_rank; /* test hook: when > 0, the sampled threshold is taken at
                                     this rank of the sample instead of the safe one (rank 1 =
                                     sample maximum, which forces the full-selection path)     */
  int32_t        nesterov;        /* 0: Algorithm 4 (vanilla momentum, Eq. 5).  1: Algorithm 5
                                     (Appendix B): U <- m*(U + g) ; V <- (V + U) + g           */
  int32_t        select_mode;     /* 0: exact top-k_j per tensor (the sample only proposes).
                                     1: Sec. 5 as stated ("paper-literal"): the threshold comes
                                     from the sample, |v| > thr is sent, at most 2 k_j entries
                                     per tensor; the count varies, see dgc_get_nnz             */
  int32_t        clip_scope;      /* 0: one clipping norm over the worker's whole gradient set
                                     (Appendix C's ||G^k||_2; the reading used everywhere else).
                                     1: every tensor is clipped by its own L2 norm against the
                                     same thr_G * N^-1/2 (Sec. 3.2 speaks of "their L2-norms");
                                     see dgc_get_clip                                          */
} dgc_config;

typedef struct dgc_status {
  double  grad_norm;          /* L2 norm of the last gradient set (0 when clipping is off)   */
  float   clip_coef;          /* coefficient applied to the last gradient (1 = not clipped)  */
  int32_t flags;              /* OR of DGC_FLAG_* over the last dgc_compress                 */
  int64_t iterations;         /* dgc_compress calls completed on the device (graph replays   */
                              /* included)                                                   */
  int64_t full_select_last;   /* tensors that took the full-selection path in the last call */
  int64_t candidates_last;    /* entries that passed the sampled thresholds in the last call */
} dgc_status;

/* Algorithm 4, line "U^k <- 0, V^k <- 0": allocates and zeroes u and v (device
 * memory of cfg->device, arena-sized), the selection scratch and the plan
 * tables.  Synchronous.  The caller's current device is the same after the
 * call as before it.  The state is owned by the caller until
 * dgc_state_destroy.  Errors: DGC_EINVAL (NULL, num_tensors < 1, numel < 1,
 * sparsity outside [0,1), sample_ratio outside [0, 0.5], select_mode or clip_scope not 0 or 1, padded arena >=
 * 2^31 elements), DGC_ENOMEM, DGC_ECUDA. */
int32_t dgc_state_create(const dgc_config* cfg, dgc_state** out);

/* Frees everything dgc_state_create allocated.  Synchronises the device. */
int32_t dgc_state_destroy(dgc_state* st);

/* Sec. 3.3 "Warm-up Training" / Sec. 4.1: change the sparsity between two
 * iterations.  Recomputes k_j = ceil(n_j (1 - s)) (integer arithmetic, parts
 * per 1e9, at least 1), the output offsets and the sampling plan, and uploads
 * them; may reallocate selection scratch.  Always synchronises the whole
 * device, before touching the state and again before returning, so work of
 * this state that is still running on any stream is waited for.  If the upload
 * fails (DGC_ENOMEM, DGC_ECUDA) the state is no longer usable: every later
 * call on it returns DGC_ESTATE until it is destroyed. */
int32_t dgc_set_sparsity(dgc_state* st, double sparsity);

/* Sec. 4.1: sparsity of warm-up stage 0..4 = 0.75, 0.9375, 0.984375, 0.996,
 * 0.999.  DGC_EINVAL for other stages.  Host only. */
int32_t dgc_warmup_sparsity(int32_t stage, double* sparsity_out);

/* Sum over tensors of k_j: the exact number of pairs every dgc_compress call
 * writes at the current sparsity.  Negative DGC_E* on error.  Host only. */
int64_t dgc_max_nnz(const dgc_state* st);

/* Host only.  Any output pointer may be NULL.
 *   arena_offset[num_tensors]   first element of tensor j in the arena
 *   k[num_tensors]              pairs emitted for tensor j per call
 *   out_offset[num_tensors + 1] tensor j's pairs are out[out_offset[j] .. out_offset[j+1])
 *   arena_len                   elements in the padded arena                          */
int32_t dgc_layout(const dgc_state* st, int64_t* arena_offset, int64_t* k, int64_t* out_offset,
                   int64_t* arena_len);

/* One iteration of Algorithm 4 on this worker, from the clipping line to the
 * end of the loop over tensors (Sec. 3.2, Eq. 5, Sec. 3.3, Sec. 5):
 *   coef = min(1, thr_G N^-1/2 / ||g||_2) over the whole set (fp64 sum), gc = g*coef
 *   u <- m*u + gc ; v <- v + u            (separately rounded fp32 operations; with
 *                                          cfg.nesterov: u <- m*(u + gc) ; v <- (v + u) + gc)
 *   per tensor j: the k_j entries of v largest in |v| (ties: lower index first)
 *   out: their (arena index, v) pairs, ascending index, at out_offset[j]
 *   v <- 0, u <- 0 at those entries (momentum factor masking)
 * A seeded sample of |v| only proposes a threshold; the result is always the
 * exact top-k_j set.  Tensors with masses of equal magnitudes (all zeros, sign
 * gradients) are completed from the tied entries of lowest index without a
 * selection (DGC_FLAG_TIE_FILL); if the proposal otherwise lets fewer than k_j or
 * too many entries pass, that tensor is selected from the whole of v instead
 * (slow, see dgc_status).
 *   grad_arena  device, const, arena_len floats, 16-byte aligned; not modified
 *   out_idx     device, capacity int32   (index into the arena)
 *   out_val     device, capacity floats
 *   capacity    >= dgc_max_nnz(st), else DGC_ECAPACITY and nothing is enqueued
 * Exactly dgc_max_nnz(st) pairs are written.  Asynchronous on `stream`; calls
 * on one state must be stream-ordered with respect to each other, and the
 * state's device must be the current device.
 * Stream capture: the call only launches kernels, and what changes from call to call
 * (the sampling seed, the bank of status counters) is derived on the device from a count
 * of completed calls kept in device memory, so the call may be captured into a CUDA graph
 * and replayed (with dgc_profile_enable off); each replay is one iteration on the buffers
 * that were captured.  dgc_get_status reports the device's count.  A graph is bound to the
 * sparsity it was captured at: capture again after dgc_set_sparsity. */
int32_t dgc_compress(dgc_state* st, const float* grad_arena, int32_t* out_idx, float* out_val,
                     int64_t capacity, void* stream);

/* dgc_compress for several workers that live on one GPU (the paper's N nodes simulated in
 * one memory): the same result as calling dgc_compress on each state in turn.  The workers'
 * kernels are spread round robin over up to 8 internal streams, forked from and joined back
 * into `stream`, so that one worker's short sampling, selection and emission kernels run
 * while other workers' streaming passes keep the memory system busy; work enqueued on `stream`
 * afterwards sees all outputs.
 *   states[num_states]  distinct states on one device;  grad_arenas, out_idx, out_val,
 *   capacity: host arrays [num_states] with the per-worker arguments of dgc_compress.
 * The internal streams and events are created on the first call for a device (make that call
 * outside stream capture) and are shared by all calls for that device: enqueue batches for one
 * device from one host thread at a time. */
int32_t dgc_compress_batch(int32_t num_states, dgc_state* const* states,
                           const float* const* grad_arenas, int32_t* const* out_idx,
                           float* const* out_val, const int64_t* capacity, void* stream);

/* The same iteration with HOST buffers: copies grad_host (arena_len floats;
 * pinned memory makes the copy asynchronous) into a staging buffer the state
 * owns (allocated on first use), runs dgc_compress, copies the dgc_max_nnz(st)
 * pairs back to out_idx_host / out_val_host and synchronises `stream`, so the
 * lists are valid on return. */
int32_t dgc_compress_host(dgc_state* st, const float* grad_host, int32_t* out_idx_host,
                          float* out_val_host, int64_t capacity, void* stream);

/* dgc_compress_host for several workers of one GPU (the same iteration of Algorithm 4 for each,
 * Sec. 3.2, Eq. 5, Sec. 3.3, Sec. 5): every worker's gradient is copied from host memory, its
 * call runs, and its dgc_max_nnz pairs are copied back, each worker on its own internal stream,
 * so that one worker's kernels run while the next worker's gradient is still crossing the bus.
 * Same results as dgc_compress_host per state.  Host arrays [num_states] of host pointers
 * (pinned memory makes the copies asynchronous); capacity[w] >= dgc_max_nnz(states[w]).
 * Synchronises `stream` before returning: the lists are valid on return.  Not for stream
 * capture (it allocates staging on first use and synchronises). */
int32_t dgc_compress_host_batch(int32_t num_states, dgc_state* const* states,
                                const float* const* grads_host, int32_t* const* out_idx_host,
                                float* const* out_val_host, const int64_t* capacity,
                                void* stream);

/* Algorithm 4, line "G_t <- sum_k encode(G~_t^k)", for N workers' lists that
 * already sit in this GPU's memory: dense_out[i] = (((+0 + val_0) + val_1) ...)
 * over the workers that list index i, in worker order, fp32; +0 elsewhere.
 * No floating-point atomics: each tile of dense_out is accumulated in shared
 * memory one worker after the other and written once.
 *   idx_lists, val_lists  host arrays [num_workers] of device pointers
 *   nnz                   host array [num_workers], pairs per list (may be 0)
 *   dense_out             device, dense_len floats, overwritten
 *   workspace             device scratch of at least
 *                         dgc_decode_workspace_bytes(num_workers, dense_len) bytes
 * Precondition: each list's indices are strictly ascending and inside
 * [0, dense_len) -- what dgc_compress produces.  A list that breaks it (a slot
 * never written, a damaged wire stream) cannot make the call write outside
 * dense_out or the workspace or read outside the lists: pairs that do not
 * belong where the order puts them are skipped, the sums of the affected
 * entries are then unspecified, and dgc_decode_rejected reports how many pairs
 * were at fault.  Such a list can also make the call slow: the work grows with
 * the sum of the upward index jumps between consecutive pairs, which is at most
 * dense_len for an ascending list but up to nnz * dense_len / 4096 steps for
 * arbitrary data.  1 <= num_workers <= DGC_MAX_DECODE_WORKERS.  Asynchronous on
 * `stream`. */
int32_t dgc_decode_accumulate(int32_t num_workers, const int32_t* const* idx_lists,
                              const float* const* val_lists, const int64_t* nnz, float* dense_out,
                              int64_t dense_len, void* workspace, int64_t workspace_bytes,
                              void* stream);
int64_t dgc_decode_workspace_bytes(int32_t num_workers, int64_t dense_len);

/* Input check of the last decode call (any of the dgc_decode_* entry points) that used
 * `workspace` with these num_workers and dense_len: synchronises `stream` and stores in
 * *rejected_out the number of pairs whose index was outside [0, dense_len) or not above its
 * predecessor in the list.  0 = the precondition held.  workspace = NULL asks about the
 * built-in scratch of dgc_decode_accumulate_static on the current device. */
int32_t dgc_decode_rejected(int32_t num_workers, int64_t dense_len, const void* workspace,
                            void* stream, int64_t* rejected_out);

/* The paper has no counterpart to this call: it is dgc_decode_accumulate for callers that
 * must not allocate device memory.  Two kinds of caller are meant.  One runs inside a
 * framework whose caching allocator has already claimed the whole GPU, so a raw cudaMalloc
 * for a workspace would fail or force the cache to be flushed.  The other sits in a
 * latency-critical loop (a serving step, a training inner loop), where cudaMalloc and cudaFree
 * are off limits because they synchronise the whole device.  Such callers still pass their
 * inputs and the output buffer, but no workspace: the tile-boundary scratch is a fixed
 * DGC_STATIC_DECODE_WORDS * 4 byte (1 MiB) array built into the library, which every GPU that
 * loads the library carries until the process exits.  The call itself performs no cudaMalloc,
 * cudaFree or other allocating call (the first call on a device looks the array up, which
 * may make the driver load the library's device code; later calls only launch kernels).
 *   Same arguments, result and preconditions as dgc_decode_accumulate (dense_out is bit for
 * bit the same), minus `workspace`.  Limit: num_workers * (ceil(dense_len / 4096) + 1025)
 * must not exceed DGC_STATIC_DECODE_WORDS (e.g. 8 workers up to 130 M dense elements); a
 * larger problem returns DGC_ECAPACITY and enqueues nothing.
 *   The first call on each device looks up the array's device address (the device that is
 * current at that call must be the one that owns the buffers).  All calls on a device share
 * the one array: it still holds the
 * previous call's boundaries, which is harmless because every word a call reads it has first
 * written itself, but two calls whose kernels overlap on the GPU (different streams, no
 * ordering) race on it and give undefined results.  Asynchronous on `stream`. */
int32_t dgc_decode_accumulate_static(int32_t num_workers, const int32_t* const* idx_lists,
                                     const float* const* val_lists, const int64_t* nnz,
                                     float* dense_out, int64_t dense_len, void* stream);

/* Algorithm 4, line "theta <- SGD(theta, G_t)" with Eq. 5's third term:
 * w[i] <- w[i] - lr * dense_grad[i], two separately rounded fp32 operations.
 * w and dense_grad are device arrays of len floats.  Asynchronous. */
int32_t dgc_apply_sgd(float* w, const float* dense_grad, int64_t len, float lr, void* stream);

/* Eq. 5, third term, applied directly: w <- w - lr * sum_k sparse(v_k) without forming
 * the dense gradient.  Only the entries of w that some worker lists change; the result is
 * bit for bit that of dgc_decode_accumulate followed by dgc_apply_sgd (the listed values are
 * summed in worker order from +0, then w[i] <- w[i] - lr * G[i]; elsewhere w - lr * (+0) = w)
 * for every finite lr >= 0; with lr infinite or NaN the dense form turns every weight into
 * NaN and this one only the listed ones, and with lr < 0 the dense form turns a weight of -0
 * into +0 where this one leaves it.
 * Arguments as for dgc_decode_accumulate, with the weight array (device, len floats, read
 * and written) in place of dense_out and the same workspace size.  Asynchronous. */
int32_t dgc_decode_apply_sgd(int32_t num_workers, const int32_t* const* idx_lists,
                             const float* const* val_lists, const int64_t* nnz, float* w,
                             int64_t len, float lr, void* workspace, int64_t workspace_bytes,
                             void* stream);

/* Sec. 3.1, encode(): 32-bit values of the entries sent plus 16-bit lengths of the zero runs
 * between them -- the wire format behind the compression ratios of Tables 3 and 4.  Entry t is
 * (runs_out[t], values_out[t]): skip runs_out[t] zeros, then store values_out[t].  More
 * than 65535 zeros in a row are bridged by filler entries (65535, +0.0f), each standing for
 * 65535 zeros and one explicit zero (the paper gives no rule for that case).  Zeros after
 * the last entry are not encoded.  Encoded size = 6 bytes per entry.
 *   idx, val      device, nnz pairs, idx strictly ascending (what dgc_compress emits)
 *   runs_out      device, capacity uint16;  values_out  device, capacity floats
 *   capacity      >= dgc_runlength_max_entries(nnz, dense_len) always suffices; below nnz
 *                 the call returns DGC_ECAPACITY and enqueues nothing; between the two,
 *                 entries beyond capacity are dropped (never written) and still counted
 *   count_out     device int64: entries the encoding has (fillers included)
 *   workspace     device, >= dgc_runlength_workspace_bytes(nnz) bytes, 8-byte aligned
 * Asynchronous on `stream`. */
int32_t dgc_encode_runlength(const int32_t* idx, const float* val, int64_t nnz,
                             uint16_t* runs_out, float* values_out, int64_t capacity,
                             int64_t* count_out, void* workspace, int64_t workspace_bytes,
                             void* stream);

/* The inverse: entry t lands at index sum_{j<t} (runs[j] + 1) + runs[t].  Writes `count`
 * (index, value) pairs, ascending (fillers come back as explicit zeros, which a sum
 * ignores), ready for dgc_decode_accumulate, and the position after the last entry to
 * *dense_len_out (device int64).  workspace >= dgc_runlength_workspace_bytes(count). */
int32_t dgc_decode_runlength(const uint16_t* runs, const float* values, int64_t count,
                             int32_t* idx_out, float* val_out, int64_t* dense_len_out,
                             void* workspace, int64_t workspace_bytes, void* stream);
int64_t dgc_runlength_max_entries(int64_t nnz, int64_t dense_len);
int64_t dgc_runlength_workspace_bytes(int64_t entries);

/* dgc_decode_accumulate and dgc_apply_sgd in one pass (Alg. 4, aggregation and update lines):
 * writes the dense gradient to dense_out exactly as dgc_decode_accumulate does and updates
 * w[i] <- w[i] - lr * dense_out[i] exactly as dgc_apply_sgd does, while the tile of the
 * gradient is still on chip (12 B/element moved instead of 16).  dense_out and w: device,
 * len floats, 16-byte aligned, distinct.  Other arguments as for dgc_decode_accumulate. */
int32_t dgc_decode_accumulate_sgd(int32_t num_workers, const int32_t* const* idx_lists,
                                  const float* const* val_lists, const int64_t* nnz,
                                  float* dense_out, float* w, int64_t len, float lr,
                                  void* workspace, int64_t workspace_bytes, void* stream);

/* Synchronises `stream`, then reports counters of the last dgc_compress. */
int32_t dgc_get_status(dgc_state* st, void* stream, dgc_status* out);

/* Entries the last dgc_compress wrote, in total and per tensor (host outputs, either may be
 * NULL).  select_mode 0: the fixed k_j, no synchronisation.  select_mode 1 (Sec. 5 taken
 * literally): synchronises `stream` and reads the counts.  In that mode every tensor j is
 * sampled: S = ceil(sample_ratio n_j) independent uniform draws (draw r at
 * floor(h n_j / 2^64), h = SplitMix64 step of (call seed xor (j << 32) xor r), call seed =
 * the same step of (cfg.seed * 0x9E3779B97F4A7C15 + calls completed)); the threshold is the
 * k_s-th largest sampled |v|, k_s = ceil(S (1 - s)); every entry with |v| > thr is sent,
 * unless more than 2 k_j pass (the reading of Sec. 5's "far more than expected"), in which
 * case the exact top-k_j is sent.  The tensors' lists are packed back to back in tensor order (ascending
 * index overall); dgc_max_nnz() is then the capacity bound sum_j min(n_j, 2 k_j), and the
 * out_offset of dgc_layout is not used. */
int32_t dgc_get_nnz(dgc_state* st, void* stream, int64_t* total_out, int64_t* per_tensor);

/* Synchronises `stream`, then copies per-tensor results of the last
 * dgc_compress to host arrays [num_tensors] (either may be NULL):
 *   kth_key     bit pattern of |v| of the smallest selected entry (the threshold of Algorithm 4)
 *   candidates  entries that passed the sampled threshold (-1: full-selection path taken) */
int32_t dgc_get_thresholds(dgc_state* st, void* stream, uint32_t* kth_key, int32_t* candidates);

/* Synchronises `stream`, then copies the clipping of the last dgc_compress to host arrays
 * [num_tensors] (either may be NULL): the L2 norm each tensor was measured by and the coefficient
 * it was scaled with (Sec. 3.2, Appendix C).  With clip_scope 0 every tensor reports the one
 * norm and coefficient of the whole set; with clipping off, 0 and 1.  With clip_scope 1,
 * dgc_status.grad_norm is the norm of the whole set and dgc_status.clip_coef the smallest
 * coefficient. */
int32_t dgc_get_clip(dgc_state* st, void* stream, double* norms, float* coefs);

/* Checkpoint / resume: copy u and v (arena_len floats each) to / from host
 * memory.  Synchronous on `stream`.  Either pointer may be NULL. */
int32_t dgc_state_read(dgc_state* st, float* u_host, float* v_host, void* stream);
int32_t dgc_state_write(dgc_state* st, const float* u_host, const float* v_host, void* stream);

/* Checkpoint / resume, the third piece of a worker's state: sets the count of completed
 * dgc_compress calls (dgc_status.iterations of the checkpointed state).  The exact top-k
 * result does not depend on it; the sample positions do, so the paper-literal mode
 * (select_mode 1) resumes bit-identically only with the count restored.  Synchronous on
 * `stream`; clears the status counters of the last call.  iterations >= 0, else DGC_EINVAL. */
int32_t dgc_state_set_iterations(dgc_state* st, int64_t iterations, void* stream);

/* Measurement aid (not part of the method): after dgc_profile_enable(st, n) the
 * next n dgc_compress calls record CUDA events on the call's stream at their
 * stage boundaries.  dgc_profile_read waits for the recorded calls and returns,
 * per call, five durations in milliseconds, ms_out[5 * call + stage]:
 *   0 clipping norm   1 sampled threshold proposal   2 streaming pass (Eq. 5
 *   update + candidate emission)   3 exact k-th key   4 ordered emission + masking
 * (`capacity` = calls ms_out has room for; *count_out = calls returned).  A
 * stage's duration includes the gap before its kernel starts.
 * dgc_profile_enable(st, 0) switches recording off. */
int32_t dgc_profile_enable(dgc_state* st, int32_t max_calls);
int32_t dgc_profile_read(dgc_state* st, float* ms_out, int32_t capacity, int32_t* count_out);

/* Measurement aid (not part of the method): where on the GPU's clock the kernels of this
 * state's calls ran, also when several states' calls overlap on different streams (which
 * events on one stream cannot show).  While enabled, every block of the sampling, streaming,
 * selection and emission kernels notes its start on the GPU's nanosecond timer.
 * dgc_timeline_read synchronises `stream` and returns, since the last read (or enable),
 *   ns_out[2 * kernel]      the earliest block start
 *   ns_out[2 * kernel + 1]  the latest block start
 * for kernel 0 sampling, 1 streaming pass, 2 selection, 3 emission (UINT64_MAX / 0 if the
 * kernel did not run), then clears them.  Differences between states on one GPU are
 * meaningful; the origin is arbitrary.  dgc_timeline_enable synchronises the device;
 * DGC_EINVAL from dgc_timeline_read if not enabled. */
int32_t dgc_timeline_enable(dgc_state* st, int32_t on);
int32_t dgc_timeline_read(dgc_state* st, void* stream, uint64_t* ns_out);

/* Number of kernels this library has launched in this process (all states). */
uint64_t dgc_launch_count(void);

const char* dgc_error_string(int32_t code);

#ifdef __cplusplus
}
#endif
#endif  /* DGC_H_ */
