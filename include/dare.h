/*
 * libdare — DARE per-layer activation-reuse attention step for bidirectional diffusion LLMs
 * on NVIDIA B200 (sm_100a).  Plain C ABI: pointers and sizes only.
 *
 * One handle = one attention layer with its reuse state (previous head-0 query, K/V cache,
 * attention-output cache, staleness counters).  One `dare_layer_step` = one denoising step of
 * that layer:
 *
 *   Alg. 1 / Alg. 2, line 1   x_norm = Norm(x)                       (RMSNorm with gain)
 *   line 2                    Q = W_Q x_norm, every token
 *   line 3 (Sec. 3.1)         s_i = 1 - cos(Q_t[i, head 0], Q_{t-1}[i, head 0])
 *   lines 4-5 (Eq. 2)         reuse set R = {i : s_i <= tau}; refresh set = complement,
 *                             emitted as an ascending, compacted index list
 *   DARE-KV (Alg. 1, Eq. 3)   K, V recomputed for the refresh set only and scattered into the cache
 *   DARE-O  (Alg. 2, Eq. 4)   attention evaluated for the refresh set's query rows only; every other
 *                             row keeps its cached attention output
 *   last line                 y = W_O O
 *   Sec. 4                    delta_i = 0 if refreshed else delta_i + 1
 *
 * Every step of that path runs in CUDA kernels of this library.  There is no CPU fallback.
 *
 * Memory and ownership
 *   - All `const void*` / `void*` arguments are DEVICE pointers unless the name ends in `_host`.
 *   - The library never allocates or frees device memory: the caller passes one workspace of
 *     `dare_layer_workspace_bytes()` bytes at creation; it holds the caches and all scratch.
 *   - Weights are borrowed for the life of the handle.  x and y belong to the caller.
 *   - Device pointers must be 16-byte aligned (DARE_ERR_ALIGN otherwise); the workspace 256-byte.
 *   - The handle itself is host memory owned by the library until `dare_layer_destroy`.
 *
 * Asynchrony
 *   `dare_layer_step` validates on the host, enqueues kernels on the given stream and returns.  The number
 *   of refreshed tokens never travels to the host during a step.  Results are valid once the caller has
 *   synchronised the stream.  The observation calls (`status`, `last_selection`, `export_state`,
 *   `import_state`, `step_host`) synchronise the stream themselves.
 *
 * Errors
 *   Status codes only; nothing is thrown, nothing aborts.  Problems seen by a kernel are recorded in a device
 *   status word that `dare_layer_status` returns: a bounded wait that ran out (every wait of a kernel on a barrier
 *   gives up after two seconds, and the kernel runs on to its normal exit), or a value of the device-side selection
 *   that failed its range check before it was used as an address (a token of the refresh list outside the step, a
 *   list length or a sequence's slice outside the list: the access is skipped and the launch goes on).  A recorded
 *   error stays until `dare_layer_clear_status`; while a time-out stands, every wait gives up at once, so results
 *   are undefined until it is cleared.
 *
 * Threading: one host thread per handle at a time.
 */
#ifndef DARE_H_
#define DARE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dare_layer dare_layer_t; /* opaque */

typedef enum {
  DARE_OK = 0,
  DARE_ERR_INVALID_ARG = 1, /* NULL pointer, bad enum, NaN threshold, struct_size mismatch */
  DARE_ERR_SHAPE = 2,       /* batch/seq/window outside the configured maxima, unsupported geometry */
  DARE_ERR_STATE = 3,       /* call not legal in the handle's current state */
  DARE_ERR_ALIGN = 4,       /* pointer alignment */
  DARE_ERR_WORKSPACE = 5,   /* workspace too small */
  DARE_ERR_CUDA = 6,        /* a CUDA runtime/driver call failed */
  DARE_ERR_TIMEOUT = 7,     /* a bounded device-side wait ran out (reported by dare_layer_status) */
  DARE_ERR_UNSUPPORTED = 8, /* configuration this build has no kernels for */
  DARE_ERR_DEVICE_CHECK = 9 /* a device-side range check failed (reported by dare_layer_status) */
} dare_status_t;

/* mode bit 0: reuse cached K/V for tokens of the reuse set (DARE-KV, Alg. 1);
 * mode bit 1: reuse cached attention outputs for them (DARE-O, Alg. 2).
 * DARE_MODE_DENSE recomputes everything but still scores and updates every cache, so that a reuse
 * step may follow (the "full dLLM" forward of Appendix E.2). */
enum { DARE_MODE_DENSE = 0, DARE_MODE_KV = 1, DARE_MODE_O = 2, DARE_MODE_BOTH = 3 };

typedef enum { DARE_F32 = 0, DARE_BF16 = 1 } dare_dtype_t;

/* kernel_path: which kernel family the handle uses. */
enum {
  DARE_PATH_AUTO = 0,   /* tcgen05/TMEM tensor-core kernels when dtype = bf16 and head_dim = 128, else SIMT */
  DARE_PATH_SIMT = 1,   /* plain fp32-accumulate CUDA-core kernels for every step (any supported geometry) */
  DARE_PATH_TENSOR = 2  /* tensor-core kernels or DARE_ERR_UNSUPPORTED */
};

typedef struct {
  uint32_t struct_size; /* sizeof(dare_layer_config_t), checked */
  int32_t d_model;      /* = n_heads * head_dim; multiple of 8 */
  int32_t n_heads;
  int32_t head_dim;     /* even; 32..256 for the SIMT path, 128 for the tensor-core path */
  int32_t max_batch;
  int32_t max_seq;
  float rope_theta;     /* rotary base (half-split pairing: element j rotates with j + head_dim/2) */
  float rms_eps;
  int32_t dtype;        /* dare_dtype_t: storage type of weights, x, y and caches; math accumulates in fp32 */
  int32_t score_head;   /* head whose query drives the drift score; the paper uses head 0 (Sec. 3.2) */
  int32_t kernel_path;  /* DARE_PATH_* */
} dare_layer_config_t;

typedef struct {
  const void* w_q; /* device, row-major [d_model (out), d_model (in)], y = W x (Alg. 1 line 2) */
  const void* w_k;
  const void* w_v;
  const void* w_o;
  const float* rms_gain; /* device, float32 [d_model] */
} dare_layer_weights_t;

/* Bytes of device workspace a layer of this configuration needs; 0 if the configuration is invalid. */
size_t dare_layer_workspace_bytes(const dare_layer_config_t* cfg);

/* Creates a layer on the current CUDA device.  Fills the rotary table inside the workspace (synchronises the
 * device once).  The first step after creation is dense whatever its mode (nothing is cached yet). */
dare_status_t dare_layer_create(const dare_layer_config_t* cfg, const dare_layer_weights_t* weights,
                                void* workspace, size_t workspace_bytes, dare_layer_t** out);

/* One denoising step (Alg. 1 when mode = KV, Alg. 2 when mode = O, both reuse rules when mode = BOTH).
 *   x, y        [batch, seq_act, d_model], dtype of the layer, covering positions
 *               [pos_begin, pos_begin + seq_act) of every sequence.
 *   threshold   tau of Eq. 2.  Negative refreshes every token, +inf reuses every token, NaN is rejected.
 *   cuda_stream a cudaStream_t (NULL = legacy default stream).
 * The first step after create/reset must have pos_begin = 0; it fixes batch and the cached extent
 * kv_len = seq_act.  Later steps may cover any window inside [0, kv_len) and must keep the same batch
 * (DARE_ERR_STATE otherwise).  Rows outside the window keep their cached K/V/O; attention always spans
 * keys [0, kv_len).
 * The call only enqueues: it neither synchronises nor allocates, and every data-dependent decision (the refresh set
 * and its size) is taken on the device.  It may therefore be captured into a CUDA graph, once a call of the same shape
 * and mode has run outside a capture (the first use of a kernel sets its attributes).  A captured step replays the
 * kernels chosen for the host-side state at capture time (first step or not, batch, kv_len), so replay it in that
 * state only; several steps per graph are worth more than one (a graph's first kernel cannot overlap the kernel
 * before it). */
dare_status_t dare_layer_step(dare_layer_t* layer, const void* x, int batch, int seq_act, int pos_begin,
                              int mode, float threshold, void* y, void* cuda_stream);

/* The same step with a threshold the step takes from its own scores (Sec. 3.1: dynamic thresholding; the reuse-rate
 * allocation of that section turns a reuse rate into the matching quantile of the drift scores, and this is that
 * quantile taken per step): the `reuse_count` tokens of the call that drifted least are reused, i.e.
 *   tau_t = the reuse_count-th smallest drift score of the step's batch * seq_act tokens,
 * and Eq. 2 is applied with it, so tokens tied with that score are reused as well.  reuse_count = 0 refreshes every
 * token, reuse_count >= batch * seq_act reuses every token; NaN scores sort last and are never reused; negative is
 * rejected.  tau_t is found on the device (an exact four-pass radix selection, one more kernel ahead of the
 * selection) and never travels to the host; dare_layer_last_threshold reads it back afterwards (the threshold of
 * the last step, whichever call gave it; synchronises the stream if the value is on the device).  A first step and
 * mode = DENSE refresh everything as always.  reuse_count = floor(phi * batch * seq_act) gives the reuse rate phi. */
dare_status_t dare_layer_step_quantile(dare_layer_t* layer, const void* x, int batch, int seq_act, int pos_begin,
                                       int mode, int reuse_count, void* y, void* cuda_stream);
dare_status_t dare_layer_last_threshold(dare_layer_t* layer, float* tau_host, void* cuda_stream);

/* Same step with HOST buffers: copies x_host to the device, runs the step, copies y back and synchronises.
 * x_host / y_host should be pinned for full copy bandwidth. */
dare_status_t dare_layer_step_host(dare_layer_t* layer, const void* x_host, int batch, int seq_act, int pos_begin,
                                   int mode, float threshold, void* y_host, void* cuda_stream);

/* The same, enqueue only: the copy in runs on a copy stream of the layer as soon as the staging buffer is free (the
 * previous step of this layer has consumed it), the step on `cuda_stream` behind it, the copy out on a second copy
 * stream behind the step; nothing else on `cuda_stream` waits for the copy out.  Steps of several layers issued this
 * way overlap one layer's copies with another's kernels (full-duplex PCIe).  x_host must stay valid and y_host is
 * defined only after dare_layer_wait_host(layer), which blocks the calling thread until the layer's last copy out
 * has landed.  The copy streams and events are created on first use and live as long as the handle. */
dare_status_t dare_layer_step_host_async(dare_layer_t* layer, const void* x_host, int batch, int seq_act, int pos_begin,
                                         int mode, float threshold, void* y_host, void* cuda_stream);
dare_status_t dare_layer_wait_host(dare_layer_t* layer);

/* Forgets every cached activation: the next step is dense and must start at position 0.  Host-only. */
dare_status_t dare_layer_reset(dare_layer_t* layer);

dare_status_t dare_layer_destroy(dare_layer_t* layer);

/* Synchronises the stream and returns the device-recorded status (DARE_OK, DARE_ERR_TIMEOUT,
 * DARE_ERR_DEVICE_CHECK) or DARE_ERR_CUDA if the stream reports an error. */
dare_status_t dare_layer_status(dare_layer_t* layer, void* cuda_stream);

/* Clears the device status word (asynchronous on the stream); the handle is usable again afterwards.  Call
 * dare_layer_reset as well if the failed step may have left the caches half written. */
dare_status_t dare_layer_clear_status(dare_layer_t* layer, void* cuda_stream);

/* Diagnostics of the error paths (nothing here faults, traps or hangs the device).
 * dare_layer_debug_wait_probe: runs the kernels' bounded wait in a one-CTA launch on a barrier that nothing ever
 *   arrives on, with `limit_ns` (at most 1e9) as its limit; the wait gives up, the launch ends normally, the status
 *   word then reads DARE_ERR_TIMEOUT.  *waited_ns_host receives how long the wait took (the call synchronises).
 * dare_layer_debug_inject: the next step overwrites, right after its selection, what = 1: the first entry of the
 *   refresh list with batch * seq_act (one past the step's tokens), what = 2: the list's length with
 *   batch * seq_act + 3; the kernels that consume the selection must flag DARE_ERR_DEVICE_CHECK and skip the access.
 *   One step only; what = 0 withdraws it. */
dare_status_t dare_layer_debug_wait_probe(dare_layer_t* layer, uint64_t limit_ns, uint64_t* waited_ns_host, void* cuda_stream);
dare_status_t dare_layer_debug_inject(dare_layer_t* layer, int what);

/* Selection of the last step, copied to host buffers (any of them may be NULL):
 *   idx_host        int32[count]  ascending flat indices b*seq_act + i of the refresh set (room for batch*seq_act)
 *   count_host      int32         |refresh set|
 *   batch_off_host  int32[batch+1] start of each sequence's slice of idx
 *   scores_host     float32[batch*seq_act] drift scores (+inf on a first step)
 *   delta_host      int32[batch*seq_act] staleness counters of the window rows (Sec. 4) */
dare_status_t dare_layer_last_selection(dare_layer_t* layer, int32_t* idx_host, int32_t* count_host,
                                        int32_t* batch_off_host, float* scores_host, int32_t* delta_host,
                                        void* cuda_stream);

/* Raw views of the caches for tests and checkpointing: copies rows [0, kv_len) of each of the first `batch`
 * sequences into host buffers shaped [batch, kv_len, d_model] (layer dtype); q_prev_host is float32
 * [batch, kv_len, head_dim].  Any pointer may be NULL. */
dare_status_t dare_layer_read_caches(dare_layer_t* layer, void* k_host, void* v_host, void* o_host,
                                     float* q_prev_host, void* cuda_stream);

/* Checkpoint / resume of the reuse state (previous query, K/V/O caches, staleness, step bookkeeping).
 * The library's own cache of projected outputs (W_O O by cache row, which lets a step with many tokens that reuses
 * attention outputs project only the refreshed rows: the paper's Alg. 2 line 11 projects every row, and a reused
 * row projects to what it projected to before) is derived data and not part of the state: after an import the next
 * steps project every row again until one of them has covered every cached row. */
size_t dare_layer_state_bytes(const dare_layer_t* layer);
dare_status_t dare_layer_export_state(dare_layer_t* layer, void* dst_host, size_t bytes, void* cuda_stream);
dare_status_t dare_layer_import_state(dare_layer_t* layer, const void* src_host, size_t bytes, void* cuda_stream);

/* Optional per-kernel timing for benchmarks: when enabled, every step records a CUDA event before each of its
 * kernels (on the step's stream).  `dare_layer_last_kernel_times` waits for the last step to finish and returns,
 * for each kernel in launch order, its slot id and the time to the next mark in milliseconds.  DARE_ERR_STATE if
 * profiling is off or no step has run since it was enabled. */
dare_status_t dare_layer_set_profiling(dare_layer_t* layer, int enable);
dare_status_t dare_layer_last_kernel_times(dare_layer_t* layer, int32_t* slot_host, float* ms_host, int capacity,
                                           int* n_out);
const char* dare_kernel_slot_name(int slot);

/* Diagnostics: when enabled, block (0,0) of each tensor-core kernel of a step writes %globaltimer values (ns) at its
 * phase boundaries into 64 slots of the workspace: slots [8k, 8k+8) belong to kernel k of the step in the order
 * Q projection, K/V projection, attention, output projection; within a kernel: start, set-up done, first operand
 * tile landed, main loop done, epilogue done, latest block start (attention with two query tiles per CTA only),
 * latest block end, blocks that ran (a running total over the steps since recording was switched on).  The
 * persistent projection kernel records start, set-up done, latest end and the count only.  After the 64 slots come
 * 1024 records (start, accumulator complete, end) of the blocks of the one-tile-per-CTA Q projection, by linear
 * block index.
 * `out_host` (may be NULL, else room for 64 + 3*1024 values) receives the buffer of the last step (the call
 * synchronises the stream); `enable` switches recording for later steps. */
dare_status_t dare_layer_debug_timestamps(dare_layer_t* layer, int enable, uint64_t* out_host, void* cuda_stream);

/* Stand-alone pieces of the path for token counts far beyond one layer step (e.g. a whole batch of sequences
 * scored at once), organised for HBM bandwidth.  Device pointers, asynchronous on the stream.
 *
 * dare_drift_scores: Sec. 3.1, s_i = 1 - cos(q_now[i], q_prev[i]) for `rows` rows of `head_dim` float32 each
 * (row-major, head_dim a multiple of 4); a zero-norm row scores 1.
 *
 * dare_select_compact: Eq. 2 and its complement over `n_tokens` float32 scores: idx receives the ascending list of
 * tokens with !(s <= threshold) (room for n_tokens entries), *count their number.  `scratch` is
 * dare_select_compact_scratch_bytes(n_tokens) bytes of device memory owned by the caller (per-tile counts and
 * offsets, and one decision bit per score: about n_tokens / 8 bytes); n_tokens <= 2^30; NaN threshold is rejected. */
dare_status_t dare_drift_scores(const float* q_now, const float* q_prev, int64_t rows, int head_dim, float* scores,
                                void* cuda_stream);
/* Alg. 1/2 line 1 alone: y[r, :] = x[r, :] / sqrt(mean(x[r, :]^2) + eps) * gain, for `rows` rows of `d_model` elements
 * (a multiple of 16) of the given dare_dtype_t; gain is float32 [d_model]; rows <= 2^24.  The kernel of the layer step. */
dare_status_t dare_rmsnorm(const void* x, const float* gain, void* y, int64_t rows, int d_model, float eps, int dtype,
                           void* cuda_stream);
/* *tau_out (device) = the k-th smallest of n_tokens float32 scores (k clamped to [0, n_tokens]; k = 0: -inf,
 * k = n_tokens or beyond the scores that are numbers: +inf), the threshold that reuses the k least-drifted tokens under
 * Eq. 2 (Sec. 3.1).  One CTA, exact; 1 <= n_tokens <= 2^24. */
dare_status_t dare_score_kth(const float* scores, int64_t n_tokens, int64_t k, float* tau_out, void* cuda_stream);
size_t dare_select_compact_scratch_bytes(int64_t n_tokens);
dare_status_t dare_select_compact(const float* scores, int64_t n_tokens, float threshold, int32_t* idx, int32_t* count,
                                  void* scratch, size_t scratch_bytes, void* cuda_stream);

/* dare_select_compact for callers that may not allocate (the paper has no counterpart: this is a service of the
 * library, not a step of the method).  An inference server that gives all device memory to its own arena at start-up,
 * or a latency-critical loop that cannot take the device-wide synchronisation of a cudaMalloc, has no scratch buffer
 * to pass; here the per-tile counts and offsets and the decision bits live in a 2 MB array inside the library image
 * (present on every GPU that loads the library until the process exits).  Same inputs, outputs and results as dare_select_compact.
 *   - n_tokens <= dare_select_compact_static_max_tokens() (= 16,777,216); more returns DARE_ERR_SHAPE.
 *   - The call allocates nothing and frees nothing, on the device or through any library.
 *   - The first call on a device looks up the array's device address (one cudaGetSymbolAddress with that device
 *     current): make that first call outside any stream capture.  The address is kept for the life of the process; a
 *     cudaDeviceReset of that device would leave it stale (do not reset a device this entry point has been used on).
 *   - All calls on a device share the array; it keeps the previous call's contents (nothing needs clearing: a call
 *     writes every entry before reading it).  Calls that overlap on the GPU, e.g. on two streams, race on it: their
 *     lists and counts are then undefined (entries may be missing, repeated or another call's), though no call ever
 *     writes outside its own idx[0, n_tokens) and count.  Serialise them (one stream, or events). */
int64_t dare_select_compact_static_max_tokens(void);
dare_status_t dare_select_compact_static(const float* scores, int64_t n_tokens, float threshold, int32_t* idx,
                                         int32_t* count, void* cuda_stream);

/* Number of kernels the last dare_layer_step enqueued (for launch accounting in benchmarks). */
int dare_layer_last_launch_count(const dare_layer_t* layer);

const char* dare_status_string(dare_status_t s);

/* Version of this ABI (bumped when a signature changes). */
int dare_abi_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DARE_H_ */
