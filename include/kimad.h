/*
 * kimad.h -- C ABI of the B200 (sm_100a) worker-side compression pass of Kimad+.
 *
 * One call of kimad_step() runs, for W independent data-parallel workers whose gradients
 * live on ONE GPU, the part of a Kimad round that sits between "gradient computed" and
 * "message uploaded" (Algorithm 1, worker lines "Select compressor" and "Upload"):
 *
 *   (a) d = grad - g                   EF21 difference (Section 3 footnote; Eq. 6)
 *   (b) err_l(k_j) = ||d_l - TopK_{k_j}(d_l)||^2 for every layer l and every candidate
 *       ratio j                        (Eq. 4; the "Errors" matrix of Algorithm 3)
 *   (c) the Kimad+ knapsack dynamic program choosing one candidate per layer so that the
 *       summed error is minimal and the summed size fits the budget c = B * t
 *                                      (Eq. 2, Eq. 3, Section 3.2, Algorithm 3)
 *   (d) TopK selection at the chosen k_l  (Section 2.2: the K entries largest in magnitude)
 *   (e) the sparse (index, value) message C(d)  (Algorithm 1, upload line)
 *   (f) g <- g + C(d)                  EF21 estimator update (Algorithm 1 aggregate line; Eq. 6)
 *
 * Beside it: the receiving side of a message and the model step (kimad_apply_packed, kimad_aggregate:
 * Algorithm 1, server lines), and, through kimad_options.policy, Kimad without layer adaptivity
 * (Section 3.1) and the error-axis reading of Algorithm 3.
 *
 * Conventions
 *   - L layers of sizes n_l, concatenated in list order into one flat vector of N elements.
 *     Worker w's vector starts at element w * worker_stride of `grads` and of `state`.
 *     The sweeps use 128-bit loads when grads, state (and est / x on the receiving side) are 16-byte aligned
 *     and worker_stride is a multiple of 4 elements; otherwise they read element by element (same results,
 *     the sweep over the gradients takes about a third longer): pad worker_stride rather than pass an odd N.
 *   - "device" pointers are CUDA device memory of the current device; "host" pointers are
 *     ordinary host memory.  The library never allocates or frees device memory: scratch is
 *     the caller's (kimad_set_workspace).  All kernels are ordered on the caller's stream (some of them
 *     run on streams of the context's own, forked from and joined to the caller's with events).
 *     grads and state of a step must not overlap and must not change while the step is in flight: the
 *     kernels re-read them instead of keeping a copy of grad - g.
 *   - TopK order inside a layer: larger |d| first (compared on the 31 magnitude bits, so +0
 *     and -0 tie), then lower index.  Inputs must be finite.
 *   - Size of a layer compressed at k: k * (4 + vb) bytes (u32 index + value of vb = 4 or 2
 *     bytes).  Budget c = floor(bandwidth * t_target) bytes.  Budget axis of the DP: D cells
 *     of c / D bytes; a candidate occupies ceil(bytes * D / c) cells.
 *   - Return values: 0 = ok; > 0 = soft status (the step ran); < 0 = error.
 */
#ifndef KIMAD_H
#define KIMAD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define KIMAD_OK 0
#define KIMAD_STATUS_INFEASIBLE 1 /* not even the smallest candidates fit: every layer took candidate 0 */
#define KIMAD_STATUS_PLATEAU 2    /* budget covers the largest candidate of every layer: all taken      */
#define KIMAD_ERR_INVALID_ARG (-1)
#define KIMAD_ERR_WORKSPACE (-2) /* workspace missing, too small or misaligned                        */
#define KIMAD_ERR_CAPACITY (-3)  /* a worker selected more entries than max_packed_elems             */
#define KIMAD_ERR_NONFINITE (-4) /* Inf/NaN met in grad - g (only reported when check_finite != 0)   */
#define KIMAD_ERR_TIMEOUT (-5)   /* reserved: no kernel of this library waits on another             */
#define KIMAD_ERR_CUDA (-6)      /* a CUDA runtime call failed                                       */
#define KIMAD_ERR_NOMEM (-7)     /* host allocation failed                                           */
#define KIMAD_ERR_TOO_LARGE (-8) /* kimad_step_builtin_scratch: scratch need above the built-in array */

#define KIMAD_MAX_RATIOS 127 /* candidates per layer */
#define KIMAD_MAX_D 8191     /* budget cells */

typedef struct kimad_ctx kimad_ctx;

typedef struct {
    uint32_t D;                 /* budget cells of the DP; 0 -> 1000 (Section 4.3: factor 1000); needs D >= L */
    uint32_t value_dtype;       /* 0: packed values are f32; 1: bf16, round-to-nearest-even          */
    uint32_t check_finite;      /* != 0: a non-finite d makes that worker's step fail with NONFINITE */
    uint32_t infeasible_policy; /* 0: take candidate 0 everywhere and report KIMAD_STATUS_INFEASIBLE */
    uint64_t max_packed_elems;  /* capacity (entries) of each worker's idx/val buffer; 0 -> N        */
    uint64_t worker_stride;     /* elements between consecutive workers in grads/state; 0 -> N; a multiple
                                   of 4 keeps the 128-bit loads (see Conventions)                     */
    uint32_t curve_mode;        /* 0: error curves from one sweep over sampled bands; a candidate whose certified
                                   bound is too loose is refined, a layer whose threshold fell outside its band
                                   takes the exact radix select; 1: exact radix select everywhere          */
    uint32_t policy;            /* 0: Kimad+, the knapsack search over the layers (Section 3.2, Algorithm 3);
                                   1: Kimad, one ratio of the grid for every layer: the largest whose total
                                      size fits c (Section 3.1; the fixed-ratio baseline of Section 4.3).
                                      A context with a single layer of N elements and policy 1 is the
                                      whole-model TopK baseline of Section 4.3 on the same grid.
                                   2: Algorithm 3 read the other way round (its header speaks of an error
                                      budget E_max and a step E_max / D): the knapsack axis is the error,
                                      e_{l,j} = floor(err_{l,j} D / E_max) cells with E_max = sum_l err_{l,0}
                                      (binary64), the value is the number of kept entries, and the answer is
                                      the lowest error level whose smallest size fits c.  Needs L * K small
                                      enough for the candidate tables to sit in shared memory (else
                                      kimad_create returns INVALID_ARG).
                                   3: Kimad as Section 3.1 states it: ONE ratio for all layers, SIZED TO THE
                                      BUDGET instead of taken from a grid: r = q / 2^32 with the largest q in
                                      [0, 2^32] such that sum_l k_l fits floor(c / (4 + vb)) entries, where
                                      k_l = min(n_l, max(1, floor(q n_l / 2^32))).  The ratio grid plays no
                                      role and must be {1.0} (n_ratios = 1); every layer has the one candidate
                                      j = 0, whose k is the fitted one (err/tau of kimad_debug_get_curve
                                      describe it; kimad_get_k_table still returns the static table, k = n_l).
                                      Fewer than one entry per layer affordable -> every k_l = 1, INFEASIBLE;
                                      everything affordable -> PLATEAU.  A context with a single layer of N
                                      elements is TopK over the whole model at K = floor(c / (4 + vb))
                                      (Section 4.3: "select K with the whole model information").            */
    uint32_t cost_model;        /* how a compressed layer is sized (Eq. 3's b_ij; the paper fixes no encoding):
                                   0: k (4 + vb) bytes, also at k = n_l;
                                   1: dense fallback: a candidate whose sparse size reaches the layer's dense size,
                                      k (4 + vb) >= vb n_l, is sent DENSELY: all n_l values in index order, no
                                      indices, vb n_l bytes; it keeps every entry and has no compression error.
                                      kimad_packed.dense flags such layers; idx is still filled (0 .. n_l - 1)
                                      so that the receiving side reads the message the same way, but a transport
                                      would not send it (used_bytes counts vb n_l).  Policies 0 and 1 only.  */
} kimad_options;

/* Per-worker result record, written by the device. */
typedef struct {
    uint64_t budget_bytes; /* c                                                          */
    uint64_t used_bytes;   /* sum of the chosen candidates' sizes (k_l (4 + vb), or vb n_l for a layer
                              sent densely under cost model 1); <= c unless status is INFEASIBLE */
    uint64_t n_selected;   /* sum_l k_l                                                  */
    float total_err;       /* err_1(k_1) + ... + err_L(k_L), added left to right in f32  */
    int32_t status;        /* 0, a KIMAD_STATUS_* or a KIMAD_ERR_* of this worker        */
} kimad_stats;

/* Output buffers of one step, all DEVICE memory owned by the caller.
 *   idx   u32 [W][max_packed_elems]  layer-local indices; layer l of worker w occupies
 *                                    [offs[w][l], offs[w][l+1]), ascending index inside a layer
 *   val   f32 or bf16 [W][max_packed_elems]  the kept d values, same positions as idx
 *   offs  u64 [W][L+1]               running sum of k_l
 *   k     u32 [W][L]                 chosen k per layer
 *   j     u32 [W][L]                 chosen candidate (index into the ratio grid) per layer
 *   stats [W]
 *   dense u32 [W][L]                 1 where the layer is sent densely (cost model 1), else 0; may be NULL */
typedef struct {
    uint32_t* idx;
    void* val;
    uint64_t* offs;
    uint32_t* k;
    uint32_t* j;
    kimad_stats* stats;
    uint32_t* dense;
} kimad_packed;

/* Problem statement of Section 3.2: the layers, the workers and the discrete ratio set
 * {c^1..c^K}.  layer_sizes: host, [n_layers], each in [1, 2^32).  ratio_grid: host,
 * [n_ratios], strictly ascending in (0, 1]; candidate k_{l,j} = min(n_l, max(1, ceil(r_j n_l))).
 * opt may be NULL (all defaults).  Host-only: touches no GPU.  *out is owned by the caller
 * until kimad_destroy.  Errors: INVALID_ARG, NOMEM. */
int kimad_create(kimad_ctx** out, const uint64_t* layer_sizes, uint32_t n_layers, uint32_t n_workers,
                 const double* ratio_grid, uint32_t n_ratios, const kimad_options* opt);
void kimad_destroy(kimad_ctx* ctx);

/* Scratch the kernels need (one code byte per element of the difference vector, histograms, tables, DP
 * back-pointers, per-chunk counts): about 1 byte per element plus about 0.4 MB per (worker, layer above 4096
 * elements). */
size_t kimad_workspace_bytes(const kimad_ctx* ctx);
/* dev_ptr: device, 256-byte aligned, at least kimad_workspace_bytes(); stays owned by the
 * caller and must outlive the context's steps.  Uploads the static tables and zeroes the
 * histograms with synchronous copies on the current device.  Errors: WORKSPACE, CUDA. */
int kimad_set_workspace(kimad_ctx* ctx, void* dev_ptr, size_t bytes);

/* One compression pass (a)-(f) for all W workers, asynchronous on cuda_stream (a cudaStream_t,
 * NULL = default stream).
 *   grads_dev  device, f32 [W][worker_stride], read only
 *   state_dev  device, f32 [W][worker_stride], the EF21 estimators g; updated in place
 *   bandwidth_bytes_per_s  host, [W]: monitored bandwidth B_m^k of each worker (Section 2.4)
 *   t_target_s one-direction communication time; budget c_w = floor(B_w * t) bytes.  A caller
 *              following Eq. 2 passes (t - T_comp) / 2; a fixed byte budget is (B = bytes, t = 1)
 *   out        host struct of device pointers (see kimad_packed)
 * Returns 0 or a CUDA/argument error; per-worker outcomes land in out->stats[w].status.
 * The step's launches, including those on the context's own streams, are ordered through events on
 * cuda_stream, so a step can be captured into a CUDA graph; the budgets are then baked into the graph. */
int kimad_step(kimad_ctx* ctx, const float* grads_dev, float* state_dev, const double* bandwidth_bytes_per_s,
               double t_target_s, const kimad_packed* out, void* cuda_stream);

/* kimad_step for callers that cannot allocate device memory.  (The paper has no counterpart: this is
 * a deployment variant of the same pass.)  Some callers have no workspace to give to
 * kimad_set_workspace and may not obtain one: a gradient hook that runs while other streams are busy
 * (cudaMalloc synchronises the whole device and would stall them), or a plug-in inside a runtime that
 * owns all device memory in a fixed arena and hands none out.  This call takes the same arguments as
 * kimad_step and produces the same results, but keeps its scratch in an array of
 * KIMAD_BUILTIN_SCRATCH_BYTES that is part of the library's device image: every GPU that loads the
 * library holds those bytes until the process exits.  It calls no cudaMalloc / cudaFree and no
 * allocating library routine; kimad_set_workspace is not needed (a workspace attached to ctx is left
 * untouched).
 *   - Limit: kimad_workspace_bytes(ctx) must not exceed KIMAD_BUILTIN_SCRATCH_BYTES, else the call
 *     returns KIMAD_ERR_TOO_LARGE and does nothing (roughly: up to a million elements over all
 *     workers with a dozen ratios).
 *   - The first call on a device looks up the array's device address (that device must be current,
 *     as for every call); make that first call before any stream capture.
 *   - All contexts and all calls on a device share the one array, which keeps the previous call's
 *     contents: every call re-uploads its tables and clears its histograms in stream order, so calls
 *     that follow each other on one stream are safe, while calls that overlap on the GPU (different
 *     streams, or different host threads) race on the scratch and must be serialised by the caller.
 *   - The kimad_debug_* getters read the attached workspace, not the built-in array. */
#define KIMAD_BUILTIN_SCRATCH_BYTES (32u << 20)
#define KIMAD_BUILTIN_MAX_DEVICES 64
int kimad_step_builtin_scratch(kimad_ctx* ctx, const float* grads_dev, float* state_dev,
                               const double* bandwidth_bytes_per_s, double t_target_s, const kimad_packed* out,
                               void* cuda_stream);

/* Copies the last step's chosen k to host_k (host, u32 [W][L]; may be NULL) after synchronising
 * cuda_stream.  Returns the most severe per-worker status of that step: the lowest negative
 * error if any worker failed, else the largest soft status, else 0. */
int kimad_get_k(kimad_ctx* ctx, uint32_t* host_k, void* cuda_stream);

/* ---- Receiving side of a message and the model step (Algorithm 1, server lines) ---------------------
 *
 * kimad_apply_packed: the receiver of the messages keeps, per sender m, a copy of that sender's
 * estimator and adds every message to it: u^_m <- u^_m + C_m(u_m - u^_m) ("Aggregate all update
 * estimators" in Algorithm 1; the same line updates the model estimator x^ on the workers when the
 * server's message is the one received).  msg: the buffers a kimad_step of a context with the SAME layer
 * list, worker count and value_dtype filled (device pointers; offs decides how many entries are read,
 * so a failed worker, whose offs are all zero, adds nothing).  est_dev: device, f32, worker w at
 * est_dev + w * worker_stride of ctx, layers concatenated as in grads; updated in place, one binary32
 * add per entry (after a step, the receiver's copy is bit-identical to the sender's state).  Entries
 * whose index is not below their layer's size are skipped.  Asynchronous on cuda_stream; the workspace
 * must be attached (it holds the layer table).  Errors: INVALID_ARG, WORKSPACE, CUDA. */
int kimad_apply_packed(const kimad_ctx* ctx, const kimad_packed* msg, float* est_dev, void* cuda_stream);

/* kimad_aggregate: the model step x <- x - gamma * sum_m w_m u^_m (last line of Algorithm 1).
 * x_dev: device f32 [n], in place.  est_dev: device f32, estimator m at est_dev + m * stride (stride
 * >= n, in elements).  weights: HOST f32 [n_workers], n_workers in [1, KIMAD_MAX_AGG_WORKERS].
 * binary32 throughout, in this order: acc = 0; acc = acc + w_m * est_m for m = 0, 1, ... (product and
 * sum rounded separately, no FMA); x = x - gamma * acc.  Asynchronous on cuda_stream; no context
 * needed.  Errors: INVALID_ARG, CUDA. */
#define KIMAD_MAX_AGG_WORKERS 64
int kimad_aggregate(float* x_dev, const float* est_dev, uint64_t stride, uint32_t n_workers, uint64_t n,
                    const float* weights, float gamma, void* cuda_stream);

/* ---- Bandwidth monitor (Section 2.4: every device estimates its bandwidth B_m^k from what it observed; the
 * paper gives no formula, this is ours).  Host-only, no GPU.  The caller reports every finished transfer (the
 * upload of a step's message: its bytes and how long it took); the estimate is the throughput over the last
 * `window` transfers, sum of bytes / sum of seconds (long transfers weigh more), smoothed exponentially:
 * est <- alpha * windowed + (1 - alpha) * est (alpha = 1: no smoothing; the first observation sets est).
 * The estimate, in bytes per second, is what kimad_step takes as bandwidth_bytes_per_s.
 *   kimad_monitor_create: window in [1, 65536], alpha in (0, 1]; errors INVALID_ARG, NOMEM.
 *   kimad_monitor_observe: seconds > 0 and finite, else INVALID_ARG (nothing recorded).
 *   kimad_monitor_estimate: 0.0 before the first observation. */
typedef struct kimad_monitor kimad_monitor;
int kimad_monitor_create(kimad_monitor** out, uint32_t window, double alpha);
void kimad_monitor_destroy(kimad_monitor* m);
int kimad_monitor_observe(kimad_monitor* m, uint64_t bytes, double seconds);
double kimad_monitor_estimate(const kimad_monitor* m);

/* Static tables (host-only calls).  host_k_table: u64 [L][K] candidates k_{l,j}. */
int kimad_get_k_table(const kimad_ctx* ctx, uint64_t* host_k_table);
/* Budget arithmetic of one worker exactly as the device applies it: c = floor(B * t); cells
 * (u64 [L][K], may be NULL) = ceil(k_{l,j} (4+vb) D / c).  Returns 0, KIMAD_STATUS_PLATEAU
 * (c covers every layer's largest candidate; cells not written) or KIMAD_STATUS_INFEASIBLE
 * (c == 0; cells not written). */
int kimad_plan_budget(const kimad_ctx* ctx, double bandwidth_bytes_per_s, double t_target_s,
                      uint64_t* budget_bytes, uint64_t* cells);

/* Stage isolation for tests.  All synchronise the device.
 * kimad_debug_get_curve: results of stage (b) of the last step; each pointer is host
 *   [W][L][K] or NULL: err (f32); shift: the threshold of the candidate is known to lie in the
 *   key interval [tau, tau + 2^shift) and to be the keep_eq-th largest key inside it.  Where
 *   shift is 0, tau is the 31-bit magnitude key of the k-th largest entry and keep_eq the number
 *   of entries equal to tau that are kept.
 * kimad_debug_get_selection: exact threshold key and number of kept ties of the candidate chosen
 *   for every layer in the last step, host u32 [W][L] each (meaningless where k = n_l or k = 0). */
int kimad_debug_get_curve(kimad_ctx* ctx, float* host_err, uint32_t* host_tau, uint32_t* host_keep_eq,
                          uint32_t* host_shift);
int kimad_debug_get_selection(kimad_ctx* ctx, uint32_t* host_tau, uint32_t* host_keep_eq);
/* kimad_step whose DP (c) consumes err_dev (device, f32 [W][L][K]) instead of the curves it
 * computed; stages (a), (b), (d)-(f) unchanged. */
int kimad_debug_step_with_err(kimad_ctx* ctx, const float* grads_dev, float* state_dev,
                              const double* bandwidth_bytes_per_s, double t_target_s, const kimad_packed* out,
                              void* cuda_stream, const float* err_dev);
/* kimad_step without stage (c): candidate j_dev[w][l] (device, u32 [W][L]) is taken as given. */
int kimad_debug_step_with_j(kimad_ctx* ctx, const float* grads_dev, float* state_dev,
                            const double* bandwidth_bytes_per_s, double t_target_s, const kimad_packed* out,
                            void* cuda_stream, const uint32_t* j_dev);

/* How many (worker, layer) pairs took the exact radix path since the workspace was attached.
 * host_count: host, u64 [6 + K]: total, then by reason: forced by curve_mode 1; bands too wide for
 * the tables; a threshold outside its sampled band; error bound too loose even after refinement; then the
 * number of pairs whose loose candidates were refined (one more pass over the layer's code bytes, not the
 * exact path); then, per candidate, how often its first bound was the loose one.  Synchronises the device. */
int kimad_debug_exact_path_layers(kimad_ctx* ctx, uint64_t* host_count);

/* Band tables of the last step, one record of four u32 per (worker, layer above the tiny size), in
 * worker-major order: bins used, entries of the cell table in use, flag (0: sampled bands in use, 1: exact
 * path forced, 2: bands did not fit the tables), detail of the misfit.  host_meta: host, u32 [W][R][4]. */
int kimad_debug_get_band_meta(kimad_ctx* ctx, uint32_t* host_meta);

/* Per-stage device timing for benchmarks.  enable != 0: every following step records CUDA events
 * around its stages on the step's stream (first use creates the events).  kimad_debug_stage_times
 * synchronises the device and writes the last step's stage durations in milliseconds to host_ms
 * (host, f32 [KIMAD_N_STAGES]), stage order: sample, sweep (difference + banded histogram), curve
 * (resolve + tiny layers), refinement and exact radix fallback, dp, select_count, select_scan, select_write. */
#define KIMAD_N_STAGES 8
int kimad_debug_enable_stage_timing(kimad_ctx* ctx, int enable);
int kimad_debug_stage_times(kimad_ctx* ctx, float* host_ms);

/* How a step schedules its workers (Section 3: every worker decides on its own, so workers are independent
 * problems).  After the sample kernel the workers are taken through the remaining stages as two groups, each on a
 * low-priority internal stream for its sweeps and a high-priority one for its short kernels (curves, DP, offsets),
 * forked from and joined to the step's stream: the short kernels of one group run beside the sweeps of the other.
 * Results do not depend on the schedule.  mode 0 (default): two groups when W >= 2 and W * N >= 2^25 elements; 1: two groups whenever
 * W >= 2; 2: one group (every kernel covers all workers, on the step's stream).  Steps with stage timing enabled
 * always run as one group. */
int kimad_debug_set_schedule(kimad_ctx* ctx, int mode);

/* kimad_step with a pair of CUDA events around every kernel launch; synchronises the device before and after and
 * writes one line per launch to text (host, text_len bytes, NUL-terminated, truncated if too short): kernel, ordinal
 * of its stream (in order of first use: 0 is the step's stream), start and end in milliseconds after the step was
 * issued.  Shows which kernels of the two worker groups run beside each other.  The events keep a kernel from being
 * scheduled ahead of its predecessor, so a traced step takes a few per cent longer than an untraced one.  A
 * development aid: one traced step at a time per process.  Arguments and errors as kimad_step. */
int kimad_debug_trace_step(kimad_ctx* ctx, const float* grads_dev, float* state_dev, const double* bandwidth_bytes_per_s,
                           double t_target_s, const kimad_packed* out, void* cuda_stream, char* text, size_t text_len);

/* Checked build of the library (compiled with -DKIMAD_CHECKED; the stand-in for a memory checker): the kernels
 * test their indices into the workspace and the output buffers before use -- a failed test sets its bit in a
 * status word and the access is skipped, nothing traps -- and the workspace regions are separated by canary words.
 * kimad_debug_check synchronises the device and reports the status word (0: no test failed since the library was
 * loaded) and the number of canaries of ctx's attached workspace that no longer hold their pattern.  Returns 1 in
 * a checked build, 0 in an ordinary build (both outputs are then 0), < 0 on error.  Either pointer may be NULL. */
int kimad_debug_check(kimad_ctx* ctx, uint32_t* failed_checks, uint32_t* damaged_canaries);

/* Kernels launched by this context so far (for launch accounting in benchmarks). */
uint64_t kimad_launch_count(const kimad_ctx* ctx);
/* Static description of a code returned by this library. */
const char* kimad_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* KIMAD_H */
