/*
 * ngc.h -- C ABI of the nested-gradient-code (NGC) hot path for NVIDIA B200 (sm_100a).
 *
 * The library simulates, on one GPU, one iteration of coded distributed gradient
 * descent with the nested gradient code of arXiv 2212.08580 ("Nested Gradient Codes
 * for Straggler Mitigation in Distributed Machine Learning"):
 *
 *   workers:    partial gradients g_j of the k data partitions (Section II-C),
 *               coded responses   x_i = b^(i) G,  X = B G      (Section II-C),
 *   main node:  choice of the component code and of the responsive set S by the
 *               progress-tracking / termination-message rule   (Sections II-D, III),
 *               decoding vector a with supp(a) in S, a B = 1   (Definition 1),
 *               decoded gradient  g = sum_{i in S} a_i x_i     (Section II-C).
 *
 * Conventions
 *   - Every function returns an int status: 0 = NGC_OK, negative = error (below).
 *     No exceptions, no abort, no device-side traps.
 *   - "host" pointers are ordinary CPU memory; "dev" pointers are CUDA device memory
 *     on the current device.  The caller owns every buffer it passes in.  The plan
 *     owns its tables and a device workspace that it allocates on first use and frees
 *     in ngc_plan_destroy.
 *   - `cuda_stream` is a cudaStream_t cast to void* (NULL = legacy default stream).
 *     Calls that take a stream only enqueue work and return; results are valid after
 *     the stream has been synchronised.  Calls on one plan must not overlap on the GPU
 *     (they share the plan's workspace).
 *   - Indices are 0-based and cyclic mod n: worker i at tolerance s holds partitions
 *     i, i+1, ..., i+s (mod n).
 */
#ifndef NGC_H
#define NGC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define NGC_MAX_N 128 /* workers */
#define NGC_MAX_S 32  /* largest straggler tolerance */
#define NGC_MAX_LEVELS 16

enum {
  NGC_OK = 0,
  NGC_ERR_INVALID = -1,     /* bad argument: sizes, ordering, null pointer, misaligned pointer, unsupported shape */
  NGC_ERR_UNDECODABLE = -2, /* more than s_L workers never finish: no component code becomes decodable */
  NGC_ERR_SINGULAR = -3,    /* decoding vector residual |a B - 1| above threshold */
  NGC_ERR_CUDA = -4,        /* a CUDA runtime call failed; see ngc_last_cuda_error */
  NGC_ERR_TIMEOUT = -5,     /* a bounded device-side wait gave up (reported by ngc_device_status) */
  NGC_ERR_NOMEM = -6,       /* host allocation failed */
  NGC_ERR_TOO_LARGE = -7    /* problem needs more scratch than the fixed array of ngc_grad_encode_static holds */
};

typedef enum { NGC_LSQ = 0, NGC_LOGISTIC = 1, NGC_SOFTMAX = 2, NGC_MLP = 3 } ngc_model_kind;
typedef enum { NGC_F32 = 0, NGC_BF16 = 1, NGC_F64 = 2 } ngc_dtype;

/*
 * The function f(d, theta) whose loss gradient is distributed (Section II-B).  The
 * paper leaves the loss open; the four kinds are least squares 1/2 (x.theta - y)^2,
 * logistic regression (labels 0/1), softmax regression (theta = W in R^{d x C},
 * row-major) and a one-hidden-layer ReLU network with softmax cross-entropy (theta =
 * [W1 (d x hidden, row-major), b1, W2 (hidden x C), b2]).  Gradients are SUMS over a
 * partition's rows (the 1/m sits in the update rule, Eq. 1).
 */
typedef struct {
  int32_t kind;               /* ngc_model_kind */
  int32_t x_dtype;            /* NGC_F32 or NGC_BF16: storage type of the data matrix */
  int32_t rows_per_partition; /* m / k */
  int32_t d;                  /* features (columns of the data matrix) */
  int32_t n_classes;          /* C, softmax / MLP only */
  int32_t hidden;             /* MLP only */
} ngc_model_t;

typedef struct ngc_plan_s ngc_plan_t; /* opaque */

/* Result of the stopping rule for one straggler pattern. */
typedef struct {
  int32_t layer;                 /* index l of the chosen component code */
  int32_t sigma;                 /* its tolerance s_l */
  int32_t nS;                    /* n - s_l */
  int32_t S[NGC_MAX_N];          /* responsive set, increasing worker index */
  double latency;                /* gamma + eps + instant the component became decodable */
  int32_t tasks_done[NGC_MAX_N]; /* partial gradients each worker had finished by then */
} ngc_step_info_t;

/* Parameter count l of a model (length of theta and of every gradient); <0 on a bad descriptor. */
int64_t ngc_num_params(const ngc_model_t *model);

/*
 * Algorithm 1 (construction of an (n, k, s_max) nested gradient code), for the listed
 * tolerances s_levels[0] < ... < s_levels[n_levels-1], each in [0, n).  Tolerance 0
 * gives B = I.  n_partitions must be a multiple of n_workers; k = q n is handled as n
 * atomic tasks of q consecutive partitions (Section II-C).  Coefficients follow the
 * cyclic-repetition scheme the paper cites: row i of B_s is supported on the window
 * i..i+s, has b_ii = 1 and lies in the null space of an s x n matrix H with zero row
 * sums whose entries are drawn from the SplitMix64 stream of `seed`.  gamma / eps are
 * the constant communication and signalling delays of Section II-D, only added to the
 * reported latency.  Pure host computation in a fixed operation order (results are
 * bit-reproducible); no GPU is touched.  *out is owned by the library.
 */
int ngc_plan(int n_workers, int n_levels, const int *s_levels, int n_partitions, uint64_t seed,
             double gamma, double eps, ngc_plan_t **out);
void ngc_plan_destroy(ngc_plan_t *plan);

/*
 * Introspection (host pointers, valid until ngc_plan_destroy).
 * ngc_plan_B: *coef points to n x (s+1) doubles, row i = B_s[i, i], B_s[i, i+1], ..., B_s[i, i+s]
 * (columns mod n); *width = s + 1.
 * ngc_plan_schedule: *order is n x (s_L+1) partition-group ids in execution order
 * (Section III, layered task scheduling); *tasks_per_layer has n_levels entries s_l + 1.
 */
int ngc_plan_B(const ngc_plan_t *plan, int layer, const double **coef, int *width);
int ngc_plan_schedule(const ngc_plan_t *plan, const int32_t **order, const int32_t **tasks_per_layer);

/*
 * Storage type of the coded gradients x_i: NGC_F64, NGC_F32, or -1 = automatic (F64
 * for least squares / logistic, F32 for softmax / MLP).  The code matrices are
 * ill-conditioned for large n and s, so F32 storage costs accuracy.
 */
int ngc_set_coded_dtype(ngc_plan_t *plan, int dtype);
int ngc_coded_dtype(const ngc_plan_t *plan, const ngc_model_t *model);

/*
 * Stopping and signalling rule (Section II-D last paragraph; Section III last
 * paragraph; proof of Theorem 1): task_times_host is n x (s_L+1) doubles, entry
 * [i][m] the duration of worker i's (m+1)-th task, +inf = never finishes.  Component
 * s_l becomes decodable when n - s_l workers have finished s_l + 1 tasks; the earliest
 * such instant wins (ties: smaller l), and exactly n - s_l responders are kept
 * (earliest first, ties by worker index).  Host only.  NGC_ERR_UNDECODABLE if no
 * component ever becomes decodable.
 */
int ngc_select(const ngc_plan_t *plan, const double *task_times_host, ngc_step_info_t *info);

/*
 * Workers' side of one iteration (Section II-C): partial gradients of all partitions
 * at theta, and the coded responses of all n workers for component `layer`.
 *   theta_dev : l floats.
 *   X_dev     : [k][rows_per_partition][d], row-major, contiguous, model->x_dtype; 16-byte aligned.
 *   y_dev     : [k][rows_per_partition]; float targets / 0-1 labels (LSQ, LOGISTIC) or int32 class ids.
 *   coded_dev : out, [n][l] in ngc_coded_dtype(plan, model); row i is x_i.
 * Each partition is read from device memory once; every g_j is computed once and fanned
 * out to the s_l + 1 workers that hold it.
 */
int ngc_grad_encode(ngc_plan_t *plan, const ngc_model_t *model, const void *theta_dev, const void *X_dev,
                    const void *y_dev, int layer, void *coded_dev, void *cuda_stream);

/*
 * Once-only preparation of the data matrix (Section II-C: the main node assigns the row blocks to the
 * workers at the beginning of training; they do not change from iteration to iteration).  Whatever the
 * library derives from the data alone is made here instead of in every ngc_grad_encode / ngc_step:
 * for NGC_MLP a bf16 copy of X_dev with a column of ones (the tensor cores' operand; device memory owned
 * by the plan, counted by ngc_workspace_bytes); nothing for the other models, whose kernels read X_dev as
 * it is.  Later calls that pass this same X_dev with the same model shape use the copy; calls with any
 * other pointer convert per call as before.  Call it again when the contents of X_dev change; X_dev =
 * NULL drops the copy.  Asynchronous on the stream (an allocation on first use aside).
 */
int ngc_prepare_data(ngc_plan_t *plan, const ngc_model_t *model, const void *X_dev, void *cuda_stream);

/*
 * Decoding vectors (Definition 1: a row of A with support in S and a B = 1), computed
 * on the device by a batched fp64 solve.  S lists responsive workers in increasing
 * order, nS >= n - s_l; if nS is larger, the n - s_l smallest indices are used, which
 * makes a unique.  a_host_out receives n doubles (zero off the used set).  Synchronous.
 * ngc_decode_vectors: `batch` patterns, S_host is batch x nS, a_host_out batch x n.
 */
int ngc_decode_vector(ngc_plan_t *plan, int layer, const int32_t *S_host, int nS, double *a_host_out);
int ngc_decode_vectors(ngc_plan_t *plan, int layer, const int32_t *S_host, int nS, int batch,
                       double *a_host_out, double *residual_host_out /* batch, may be NULL */);

/*
 * Main node's decode (Section II-C): g = sum_{i in S} a_i x_i with a from the solve
 * above.  coded_dev is [n][l] as written by ngc_grad_encode for the same layer;
 * grad_dev receives l floats.  Asynchronous on the stream.
 */
int ngc_decode(ngc_plan_t *plan, int layer, const int32_t *S_host, int nS, const void *coded_dev,
               int coded_dtype, int64_t l, float *grad_dev, void *cuda_stream);

/*
 * One full iteration for a given straggler pattern: ngc_select on the host, then
 * ngc_grad_encode for the chosen component and ngc_decode over its responsive set,
 * enqueued on the stream.  coded_dev is caller-provided scratch of n x l coded values; it
 * holds the workers' coded gradients x_i afterwards, as ngc_grad_encode would leave them.
 * The responsive set is known before any gradient is, so the decoding vector is solved on
 * a stream of the plan's own while the gradients are computed, and for the softmax and
 * MLP models the weighted sum of the decode is formed by the encode kernel from the coded
 * values as it writes them (same result as ngc_decode up to the order of its fp64 sums).
 * The first call for a model allocates the plan's scratch (ngc_workspace_bytes).
 */
int ngc_step(ngc_plan_t *plan, const ngc_model_t *model, const void *theta_dev, const void *X_dev,
             const void *y_dev, const double *task_times_host, void *coded_dev, float *grad_dev,
             ngc_step_info_t *info, void *cuda_stream);

/*
 * Same iteration with every buffer in HOST memory: copies theta, X, y to the device,
 * runs ngc_step, copies the decoded gradient back and synchronises.  Device staging
 * buffers belong to the plan and are reused across calls.
 */
int ngc_step_host(ngc_plan_t *plan, const ngc_model_t *model, const float *theta_host, const void *X_host,
                  const void *y_host, const double *task_times_host, float *grad_host, ngc_step_info_t *info);

/*
 * One problem sharded over several GPUs (Section II-C: the data is split into row blocks that independent
 * workers hold; here a GPU holds a contiguous block of partition groups and simulates the workers that start
 * in it).  A rank calls, per iteration:
 *   1. ngc_shard_gradients on its own partitions: G_dev[j] = g_j for its n_local groups (fp32, row stride ld
 *      >= l, a multiple of 4; X_local_dev / y_local_dev point at the rank's first partition and hold
 *      n_local * q partitions);
 *   2. (caller) fetches the partial gradients of the next s_l groups in cyclic order from the ranks that
 *      own them and appends them: G_window_dev = [own n_local rows; s_l halo rows];
 *   3. ngc_shard_encode_decode: the coded gradients x_i of workers first_worker .. first_worker + n_local - 1
 *      (coded_dev rows 0 .. n_local - 1; it needs room for n_local + s_l rows, the rest is scratch), and this
 *      rank's share of the decode, sum over its responsive workers of a_i x_i with a the decoding vector of
 *      the WHOLE responsive set S_host (every rank passes the same S).  partial_dev receives l values in the
 *      coded dtype, unrounded when that is fp64: the code is ill-conditioned, the shares are large and
 *      cancel, so they are added across ranks before anything is rounded to fp32;
 *   4. (caller) one all-reduce (sum) of partial_dev over the ranks gives the decoded gradient.
 * Results equal those of ngc_grad_encode + ngc_decode on one GPU up to summation order.  n_local + s_l <=
 * NGC_MAX_N.  Asynchronous on the stream, except that the first step-3 call for a (level, first_worker, n_local)
 * uploads that shard's rows of the code matrix after waiting for the stream (a rank asks for the same shard in
 * every iteration, so this happens once per level; such a call cannot be captured into a graph).
 * ngc_shard_prepare_data is ngc_prepare_data for a shard: X_local_dev holds the rank's n_local * q partitions.
 */
int ngc_shard_prepare_data(ngc_plan_t *plan, const ngc_model_t *model, const void *X_local_dev, int n_local,
                           void *cuda_stream);
int ngc_shard_gradients(ngc_plan_t *plan, const ngc_model_t *model, const void *theta_dev, const void *X_local_dev,
                        const void *y_local_dev, int n_local, float *G_dev, int64_t ld, void *cuda_stream);
int ngc_shard_encode_decode(ngc_plan_t *plan, const ngc_model_t *model, int layer, int first_worker, int n_local,
                            const float *G_window_dev, int64_t ld, const int32_t *S_host, int nS, void *coded_dev,
                            void *partial_dev, void *cuda_stream);

/*
 * Gradient-descent update of Eq. 1: theta <- theta - step * g with step = eta_t / m (the 1/m of Eq. 1 is
 * the caller's: the decoded gradient is a plain sum).  theta_dev and grad_dev hold l floats; asynchronous
 * on the stream, so it can be enqueued right behind ngc_step.
 */
int ngc_gd_update(float *theta_dev, const float *grad_dev, int64_t l, float step, void *cuda_stream);

/*
 * Response-time model of Section II-D (Eq. 2 without the constants): task_times_host
 * [n][tasks] = shift + Exp(rate) i.i.d. from the SplitMix64 stream of `seed`; each
 * worker fails (all entries +inf) independently with probability p_fail.  Host only.
 */
int ngc_sample_times(uint64_t seed, int n, int tasks, double shift, double rate, double p_fail,
                     double *task_times_host);

/*
 * Variant of ngc_grad_encode (least squares and logistic only) that allocates NO device memory.
 * (The paper has no counterpart: this is a property of the library, not of the method.)
 *
 * It is meant for callers that cannot call cudaMalloc at this point of their program: a process
 * whose GPU memory has been handed over completely to its own pool allocator, so that a raw
 * allocation would fail or fragment that pool, or a latency-critical loop that cannot take the
 * device-wide stall an allocation or a free may cause.  The scratch that ngc_grad_encode takes
 * from the plan (per-CTA partial gradients, a device copy of the component code's coefficients, a
 * status word) lives instead in one fixed array of NGC_STATIC_SCRATCH_BYTES inside the library
 * image; every GPU that loads the library holds that much until the process exits.
 *
 * Arguments are those of ngc_grad_encode; the plan is only read (its host tables), so a plan that
 * has never touched the GPU works.  status_dev may be NULL; if given, it points to one int32 in
 * device memory that is cleared by the call and set to 1 if a bounded device-side wait gave up.
 * That word is the only place where such a timeout shows: without it the flag stays inside the
 * array, and ngc_device_status, which reads the plan's own word, does not see this entry point.
 * Limit: n * slots * d * 4 bytes of partial gradients must fit in 8 MiB, where slots is the largest
 * number of CTAs that share one partition group (about 148 / n + 2 on a B200); larger problems are
 * refused with NGC_ERR_TOO_LARGE before anything is enqueued.
 * The first call on each device looks up the array's device address (with that device current);
 * make that first call before any stream capture begins.  All calls, from every plan and stream,
 * share the one array: two calls that overlap on the GPU race on it, so keep them ordered.  The
 * array keeps the previous call's contents; the call clears the status word itself and writes
 * every scratch slot before reading it.
 */
#define NGC_STATIC_SCRATCH_BYTES (256 + NGC_MAX_N * (NGC_MAX_S + 1) * 8 + 8 * 1024 * 1024)
int ngc_grad_encode_static(const ngc_plan_t *plan, const ngc_model_t *model, const void *theta_dev,
                           const void *X_dev, const void *y_dev, int layer, void *coded_dev,
                           int32_t *status_dev, void *cuda_stream);

/*
 * Latency analysis of Section IV.
 * ngc_latency_cdf_gc: Lemma 2, P(T_GC <= t) of an (n, k, sigma) gradient code.
 * ngc_latency_cdf_ngc: Theorem 1, P(T_NGC <= t) of the fully nested (n, k, s_max) code (components 0..s_max).
 * Per-task time = rho + Exp(lambda); gamma / eps the constant delays; workers fail independently with p_fail.
 * Host only.  They return a negative number on invalid arguments.
 * ngc_latency_mc: the same quantity by simulation for ANY plan: `trials` straggler patterns are drawn on the
 * device (trial r uses the ngc_sample_times stream of seed SplitMix64(seed ^ 0xD1B54A32D192ED03, r + 1)), run
 * through the stopping rule, and the latency (plan's gamma + eps + decode instant; +inf when no component ever
 * becomes decodable) and the chosen level (-1 when none) are written to latency_dev[trials] / level_dev[trials]
 * (device memory; one of the two may be NULL, not both).  Asynchronous on the stream.
 */
double ngc_latency_cdf_gc(int n, int sigma, double t, double lambda, double rho, double gamma, double eps,
                          double p_fail);
double ngc_latency_cdf_ngc(int n, int s_max, double t, double lambda, double rho, double gamma, double eps,
                           double p_fail);
int ngc_latency_mc(ngc_plan_t *plan, uint64_t seed, int64_t trials, double rho, double lambda, double p_fail,
                   double *latency_dev, int32_t *level_dev, void *cuda_stream);

/*
 * Timing of the dominant kernel of ngc_grad_encode (the fused gradient kernel).  While enabled,
 * every ngc_grad_encode call brackets that kernel with CUDA events on the launching stream.
 * ngc_profile_read synchronises those events, returns their summed elapsed milliseconds and the
 * number of bracketed launches since the last read, and resets both.
 */
int ngc_profile_enable(ngc_plan_t *plan, int on);
int ngc_profile_read(ngc_plan_t *plan, double *ms_total_out, int64_t *launches_out);

/* Bytes of device workspace the plan currently holds. */
size_t ngc_workspace_bytes(const ngc_plan_t *plan);
/* Synchronises the device and returns NGC_OK or NGC_ERR_TIMEOUT / NGC_ERR_SINGULAR from the status
 * words the kernels of this plan wrote; *residual_out (may be NULL) gets the largest decode residual seen.
 * A timeout is reported once: the call that returns NGC_ERR_TIMEOUT clears the word, so that the plan can
 * be used, and judged, again. */
int ngc_device_status(ngc_plan_t *plan, double *residual_out);
/*
 * Self-test of the failure path of the device-side waits (a property of the library; the paper has no
 * counterpart).  Every wait of a kernel on a copy or on the tensor cores is bounded: after a cycle limit
 * the kernel sets the plan's status word and returns instead of spinning.  This call enqueues one warp
 * that waits at most limit_cycles (1 .. 2e9) SM cycles on a barrier that nothing will ever complete and
 * then takes exactly that exit.  Afterwards ngc_device_status returns NGC_ERR_TIMEOUT (once), and the
 * plan and the CUDA context remain usable.  Nothing faults or hangs.
 */
int ngc_selftest_wait_timeout(ngc_plan_t *plan, int64_t limit_cycles, void *cuda_stream);
/*
 * Introspection for tests (host only, no GPU needed; a property of the library, the paper has no
 * counterpart).  The backward contractions of the dense models on CTA pairs (softmax: G_j = X_j^T R_j with the
 * 256 classes on the M side; MLP: [dW1; db1] = [X 1]^T delta1 with the hidden units on the M side in
 * `m_blocks` blocks of 256) cut the `n_cols` columns of the other operand into passes of 512 columns, may
 * cut some passes into halves of 256 to even out the load, and deal these units to at most `max_pairs`
 * CTA pairs.  This call returns that unit list for a problem of `batch` partitions and `k_chunks` chunks of
 * 64 rows per partition: row u of units_out (caller-owned host array of cap rows x 8 int32) gets
 * {pair, round, partition, M block, first column, width, first column, width} of the u-th unit in the order
 * the pairs take them; a second width of 0 means the unit has one column range.  Widths are multiples of
 * 32 and at most 256; ranges may run past n_cols (those columns are neither read nor stored).
 * *n_units_out gets the number of units (which may exceed cap: then only cap rows were written),
 * *n_pairs_out the number of pairs.  NGC_ERR_INVALID for non-positive sizes or NULL outputs.
 */
int ngc_dense_schedule(int batch, int m_blocks, int n_cols, int k_chunks, int max_pairs, int32_t *units_out, int cap,
                       int *n_units_out, int *n_pairs_out);
/* cudaError_t of the last failed runtime call on this plan (0 if none). */
int ngc_last_cuda_error(const ngc_plan_t *plan);
/* How many kernels of this library the plan has launched so far. */
int64_t ngc_launch_count(const ngc_plan_t *plan);
const char *ngc_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* NGC_H */
