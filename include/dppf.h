/*
 * dppf.h -- C ABI of the DPPF communication-round consensus step on one GPU.
 *
 * The M worker replicas of a d-parameter model live in one device buffer
 * x[M, ld] (fp32, row-major, row m = worker m).  One round
 *   1. forms the average x_A = (1/M) sum_m x_m            (Algorithm 1, last line),
 *   2. measures r_m = ||x_m - x_A||_2 for every worker     (norm in the single-line
 *      update, Sec. 5; the consensus distance logged in the ablations),
 *   3. applies x_m <- x_m + (x_A - x_m)(alpha - lambda / r_m) to every replica,
 *      all workers using the same pre-round x_A            (single-line pull-push
 *      update, Sec. 5; first display of the proof of Theorem 1).
 * x_A is never stored: it is recomputed per tile in registers.
 *
 * Conventions for every entry point
 *   - Pointers named x, v, g, norms_out, ws, x_dev are DEVICE pointers owned by the
 *     caller; *_host pointers are HOST pointers.  The library allocates nothing
 *     (dppf_consensus_static keeps its scratch in a fixed array inside the library).
 *   - Layout: row stride ld >= d with ld % 32 == 0, base pointers 128-byte
 *     aligned, so every row starts on a 128-byte boundary (a stride that is a
 *     multiple of 64 floats, i.e. 256 bytes, measures 1-3 % faster).  Columns d..ld-1
 *     are never read into a result and never written.
 *   - Updates are in place and asynchronous on `cuda_stream` (a cudaStream_t cast
 *     to void*; NULL = the legacy default stream).  Calls that touch the same
 *     buffers or the same workspace must be ordered on one stream.
 *   - x, v and g must not overlap.
 *   - Scalars are fp32 and must be finite; alpha outside (0,1] and negative
 *     lambda are accepted (the invariants alpha = 0 and lambda = 0 need them).
 *   - Return value: a dppf_status.  Arguments are checked before any CUDA call: on
 *     DPPF_ERR_INVALID_ARG, _ALIGNMENT or _WORKSPACE nothing has been launched and no
 *     buffer has been touched.
 *   - Zero distance (r_m == 0, e.g. M == 1 or identical replicas): the paper
 *     leaves 0/0 undefined; here no push is applied, the replica is left
 *     bit-for-bit unchanged and r_m = 0 is reported.
 *   - Results are run-to-run reproducible on a given GPU model for a given kernel schedule:
 *     the tile-to-block map is static and every reduction runs in a fixed order (no float
 *     atomics).  Different schedules (DPPF_PATH_*) group the sums of squares differently and
 *     may differ in the last bits of r_m and hence of x.  A call whose cooperative launch the
 *     runtime refuses falls back to a two-launch schedule (see dppf_consensus_ex); a caller
 *     that needs bit-identical repeats under such conditions asks for DPPF_PATH_TWO_KERNEL.
 *   - Accuracy against the definition evaluated in fp64: r_m to 1e-5 relative (fp32 squares
 *     summed in short fp32 runs, then fp64); every updated element to 1e-6 (1 + |x|) for
 *     replicas that lie close together compared with their magnitude and a push of the order
 *     of the distances, the regime of trained replicas.  x_m + (x_A - x_m) c_m is formed in fp32
 *     from x_m and c_m (x_A - x_m), so its error is about one fp32 ulp of the larger of the two
 *     terms: when the replicas are as far apart as they are large, or lambda / r_m is large
 *     (a push much longer than the distances), allow 1.5e-7 max(|x_m|, |step|) on top.
 */
#ifndef DPPF_H
#define DPPF_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DPPF_OK = 0,
    DPPF_ERR_INVALID_ARG = 1,  /* null pointer, M/d/ld out of range, non-finite scalar, overlap */
    DPPF_ERR_ALIGNMENT = 2,    /* base pointer not 128-byte aligned or ld % 32 != 0 */
    DPPF_ERR_WORKSPACE = 3,    /* ws_bytes < dppf_workspace_bytes(M, d) */
    DPPF_ERR_CUDA = 4,         /* a CUDA runtime call or launch failed */
    DPPF_ERR_TIMEOUT = 5       /* device status only: a bounded wait on an async copy gave up */
} dppf_status;

/* Largest worker count handled (rows of x).  The kernels are built for the worker counts the
 * paper runs (4 and 8) and up to 16: those stream at about the device's copy rate.  Above 16
 * a simpler kernel family keeps the call correct but reaches only 0.2-0.5 of that rate. */
#define DPPF_MAX_WORKERS 1024

/* Kernel schedule selector for the *_ex entry points. */
#define DPPF_PATH_AUTO 0        /* library picks */
#define DPPF_PATH_TWO_KERNEL 1  /* distance pass, then update pass, as two launches */
#define DPPF_PATH_COOPERATIVE 2 /* one persistent cooperative launch with a grid-wide barrier */
#define DPPF_PATH_STAGED 3      /* cooperative launch, rows staged through shared memory by bulk
                                   async copies; what AUTO picks for dppf_consensus when M <= 16 */

/*
 * Scratch size in bytes for a round on M replicas of length d (the per-block
 * partial sums of squared distances of step 2, plus a small header).  Returns 0
 * for invalid M or d.  The workspace needs no initialisation and may be reused
 * by later calls on the same stream.
 */
size_t dppf_workspace_bytes(int M, int64_t d);

/*
 * One pull-push round in place on x[M, ld] (steps 1-3 above; Sec. 5 single-line
 * update with x_C = x_A).  norms_out: NULL, or device fp32[M] that receives the
 * PRE-update distances r_m (the consensus distance the paper logs per worker).
 */
int dppf_consensus(float *x, int M, int64_t d, int64_t ld, float alpha, float lambda,
                   float *norms_out, void *ws, size_t ws_bytes, void *cuda_stream);

/* Same, with an explicit kernel schedule (DPPF_PATH_*).  Every schedule is reproducible
 * run to run; TWO_KERNEL and COOPERATIVE agree bit for bit, STAGED groups the sums of
 * squares differently and may differ from them in the last bits of r_m.  If the runtime
 * refuses a cooperative launch (its blocks cannot all be resident, e.g. SMs shared with
 * another client) the call falls back to the two-launch schedule; dppf_device_schedule
 * tells which schedule ran. */
int dppf_consensus_ex(float *x, int M, int64_t d, int64_t ld, float alpha, float lambda,
                      float *norms_out, void *ws, size_t ws_bytes, int path, void *cuda_stream);

/*
 * One worker's share of a round when every GPU holds ONE replica, the arrangement the paper
 * itself runs (Algorithm 1: the workers obtain the consensus variable with one collective per
 * round, then each pulls and pushes its own replica; Sec. 5 single-line update):
 *   x          device fp32[d], 128-byte aligned: this worker's replica, updated in place
 *   x_reduced  device fp32[d], 128-byte aligned: the all-reduced parameters of all workers;
 *              x_A = scale * x_reduced (scale = 1/M after a sum all-reduce, 1 after a mean)
 *   norm_out   NULL, or device fp32[1]: r = ||x - x_A|| before the update
 *   r <- ||x - x_A||,  x <- x + (x_A - x)(alpha - lambda / r);  r == 0 leaves x untouched.
 * The collective is the caller's (e.g. an NCCL all-reduce of the d floats on the same stream,
 * issued before this call); no second exchange is needed, because each worker's norm only
 * involves its own replica and x_A.  One cooperative launch (two launches if refused),
 * 5 d 4 bytes of traffic.  ws: dppf_workspace_bytes(1, d).  x, x_reduced, ws must not overlap.
 */
int dppf_worker_update(float *x, const float *x_reduced, float scale, int64_t d, float alpha,
                       float lambda, float *norm_out, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * n_rounds pull-push rounds back to back on x[M, ld], as ONE device pass sequence: the
 * single-line update of Sec. 5 applied n_rounds times, every round from its own pre-round
 * average (proof of Theorem 1, first display; the noise-free iteration whose distances the
 * theorem follows to lambda/alpha).  The result is that of n_rounds calls of
 * dppf_consensus up to the grouping of the sums of squares (last bits of r_m), but the
 * update pass of round k also accumulates the squared distances of round k+1 from the values
 * it has just formed, so the call moves (1 + 2 n_rounds) M d 4 bytes instead of
 * 3 n_rounds M d 4 and needs one launch per 256 rounds.
 *   lambdas_host  HOST fp32[n_rounds] with the push strength of every round (e.g. from
 *                 dppf_lambda_schedule), or NULL: every round uses `lambda`.
 *   norms_out     NULL, or device fp32[n_rounds, M]: row k receives the distances r_m before
 *                 round k (the per-round consensus distances the ablations plot).
 * Workspace and layout rules as for dppf_consensus.  M <= 16 runs the fused schedule; M = 1 and
 * M > 16, and any M when the runtime refuses a cooperative launch, run one round per launch
 * instead (same results, 3 M d 4 bytes per round).  The _ex form selects the kernel family:
 * DPPF_PATH_STAGED (default), DPPF_PATH_COOPERATIVE (register kernel),
 * DPPF_PATH_TWO_KERNEL (one round per call of dppf_consensus_ex).
 * If a bounded wait gives up (dppf_device_status: DPPF_ERR_TIMEOUT) x is untouched when that
 * happened before the first update and holds a mixture of rounds otherwise.
 */
int dppf_consensus_rounds(float *x, int M, int64_t d, int64_t ld, float alpha, float lambda,
                          const float *lambdas_host, int n_rounds, float *norms_out, void *ws,
                          size_t ws_bytes, void *cuda_stream);
int dppf_consensus_rounds_ex(float *x, int M, int64_t d, int64_t ld, float alpha, float lambda,
                             const float *lambdas_host, int n_rounds, float *norms_out, void *ws,
                             size_t ws_bytes, int path, void *cuda_stream);

/*
 * One round split at its reduction, for replicas whose COLUMNS are sharded over several GPUs
 * (each GPU holds x[M, d_g]: all M workers, a slice of the parameters).  In Algorithm 1 the
 * workers meet once per round to "obtain x_C"; with column shards the average of a column is
 * local to the GPU that holds it, and what has to be exchanged instead is the M sums of squares
 * behind the norms ||x_m - x_A|| of the single-line update (Sec. 5):
 *   dppf_distance_partials   sums_out[m] = sum over this shard's columns of (x_m - x_A)^2
 *                            (device fp64[M]; deterministic: fixed block order);
 *   -- the caller adds the M doubles over all shards (e.g. an all-reduce) --
 *   dppf_update_from_sums    r_m = sqrt(sums[m]), c_m = alpha - lambda / r_m, then the update
 *                            x_m <- x_m + (x_A - x_m) c_m on this shard (sums: device fp64[M],
 *                            the TOTALS over all shards; norms_out: NULL or device fp32[M], r_m).
 * With one shard the pair equals dppf_consensus (two-launch schedule) bit for bit.  A worker
 * with sums[m] == 0 is left untouched.  dppf_distance_partials reads x only; its workspace is
 * that of dppf_consensus.  dppf_update_from_sums needs no workspace.  Any M <= DPPF_MAX_WORKERS.
 * A shard may be a column range of a wider buffer (pointer x + first column, same ld).
 */
int dppf_distance_partials(const float *x, int M, int64_t d, int64_t ld, double *sums_out, void *ws,
                           size_t ws_bytes, void *cuda_stream);
int dppf_update_from_sums(float *x, int M, int64_t d, int64_t ld, float alpha, float lambda,
                          const double *sums, float *norms_out, void *cuda_stream);

/*
 * General consensus round (Algorithm 1 with an arbitrary consensus variable; Sec. 5,
 * step (a) of the regulariser-gradient equation; the remark on LSGD in the appendix):
 *   x_C  = sum_m w_m x_m / sum_m w_m      weights_host: HOST fp32[M], NULL = all equal (x_C = x_A);
 *                                         a one-hot vector makes one worker the leader
 *   y_m  = (1 - alpha) x_m + alpha x_C    pull line of Algorithm 1
 *   u_m  = (y_m - P) / ||y_m - P||        push line of Algorithm 1, P = x_A
 *                                         (DPPF_PUSH_FROM_AVERAGE) or P = x_C
 *                                         (DPPF_PUSH_FROM_CONSENSUS: push opposes the leader)
 *   x_m <- y_m + lambda u_m                                     two_term == 0
 *   x_m <- y_m + lambda (u_m - (1/M) sum_j u_j)                 two_term != 0: both terms of
 *                                         the gradient of the relaxed Inverse-Mean-Valley
 *                                         regulariser, lambda = lambda_r / M
 * x_A, x_C and P are the pre-round values for every worker.  A worker whose pulled point
 * equals P has no direction and is not pushed (with equal weights x_C is x_A bit for bit, so
 * alpha = 1 with the push taken from the average puts every replica on x_A, to fp32 rounding,
 * and reports zero push distances).  With weights_host == NULL, push from the
 * average, two_term == 0 and alpha < 1 this is dppf_consensus.  Identical replicas are left
 * untouched.  M <= 16.  norms_out (device fp32[M] or NULL) receives ||x_m - x_A|| before the
 * round, push_norms_out (device fp32[M] or NULL) receives ||y_m - P||.  Workspace and layout
 * rules as for dppf_consensus; same traffic (two reads and one write of x).
 */
#define DPPF_PUSH_FROM_AVERAGE 0
#define DPPF_PUSH_FROM_CONSENSUS 1
int dppf_consensus_general(float *x, int M, int64_t d, int64_t ld, float alpha, float lambda,
                           const float *weights_host, int push_from, int two_term,
                           float *norms_out, float *push_norms_out, void *ws, size_t ws_bytes,
                           void *cuda_stream);
/* Same with an explicit schedule: DPPF_PATH_AUTO or DPPF_PATH_STAGED (one cooperative launch,
 * rows staged through shared memory; falls back to two launches if the runtime refuses it) or
 * DPPF_PATH_TWO_KERNEL (distance launch, then update launch, register kernels).  The two
 * schedules group the sums of squares differently (last bits of the distances). */
int dppf_consensus_general_ex(float *x, int M, int64_t d, int64_t ld, float alpha, float lambda,
                              const float *weights_host, int push_from, int two_term,
                              float *norms_out, float *push_norms_out, void *ws, size_t ws_bytes,
                              int path, void *cuda_stream);

/*
 * One local optimiser step between rounds, in place, for all M workers
 * (Algorithm 1, the local update line; the experiments run SGD with momentum
 * and weight decay, whose recurrence the paper does not print -- the coupled
 * form is used):   g~ = g + weight_decay * x ;  v <- momentum * v + g~ ;
 *                  x <- x - lr * v.
 * v[M, ld] is the momentum buffer (0 before the first step), g[M, ld] the
 * gradients (read only).  Same layout rules as x.
 */
int dppf_local_step(float *x, float *v, const float *g, int M, int64_t d, int64_t ld,
                    float lr, float momentum, float weight_decay, void *cuda_stream);

/*
 * The last local step before a round fused with the round: exactly
 * dppf_local_step followed by dppf_consensus, but the distance pass reads x, v, g
 * once and produces the stepped replicas and their distances together.
 */
int dppf_local_step_and_consensus(float *x, float *v, const float *g, int M, int64_t d,
                                  int64_t ld, float lr, float momentum, float weight_decay,
                                  float alpha, float lambda, float *norms_out, void *ws,
                                  size_t ws_bytes, void *cuda_stream);

/* With an explicit schedule.  AUTO picks DPPF_PATH_STAGED for M <= 8 (x, v and g streamed
 * through shared memory in the step-and-distance pass, the plain staged update pass after the
 * grid barrier) and DPPF_PATH_COOPERATIVE (register kernel) above.  The fused call rewrites x
 * and v in its first pass already, so after a DPPF_ERR_TIMEOUT status they are partly stepped. */
int dppf_local_step_and_consensus_ex(float *x, float *v, const float *g, int M, int64_t d,
                                     int64_t ld, float lr, float momentum, float weight_decay,
                                     float alpha, float lambda, float *norms_out, void *ws,
                                     size_t ws_bytes, int path, void *cuda_stream);

/*
 * AdamW as the local optimiser (the paper's ViT runs: AdamW, lr 5e-4, weight decay 0.01;
 * appendix, "Experiments with ViT").  The recurrence is not printed in the paper; the
 * decoupled-weight-decay form is used, step = t >= 1 counting this step:
 *   x <- x (1 - lr wd);  m <- beta1 m + (1 - beta1) g;  v <- beta2 v + (1 - beta2) g^2;
 *   x <- x - lr (m / (1 - beta1^t)) / ( sqrt(v / (1 - beta2^t)) + eps )
 * exp_avg (m) and exp_avg_sq (v) are device [M, ld] buffers, zero before step 1; g is read
 * only; x, exp_avg, exp_avg_sq, g must not overlap; 0 <= beta < 1.
 * dppf_adamw_step: the step alone, any M <= DPPF_MAX_WORKERS (7 x M d 4 bytes of traffic).
 * dppf_adamw_step_and_consensus: the last step before a round fused with the round's
 * distance pass (M <= 16; 9 x M d 4 bytes instead of 7 + 3): identical to dppf_adamw_step
 * followed by dppf_consensus up to the grouping of the sums of squares.
 */
int dppf_adamw_step(float *x, float *exp_avg, float *exp_avg_sq, const float *g, int M, int64_t d,
                    int64_t ld, float lr, float beta1, float beta2, float eps, float weight_decay,
                    int step, void *cuda_stream);
int dppf_adamw_step_and_consensus(float *x, float *exp_avg, float *exp_avg_sq, const float *g, int M,
                                  int64_t d, int64_t ld, float lr, float beta1, float beta2, float eps,
                                  float weight_decay, int step, float alpha, float lambda,
                                  float *norms_out, void *ws, size_t ws_bytes, void *cuda_stream);
/* Same with an explicit schedule: DPPF_PATH_AUTO / DPPF_PATH_COOPERATIVE (one persistent launch:
 * step + distance pass, grid barrier, update pass; falls back to two launches if the runtime
 * refuses it) or DPPF_PATH_TWO_KERNEL.  Both schedules use the same grid and agree bit for bit. */
int dppf_adamw_step_and_consensus_ex(float *x, float *exp_avg, float *exp_avg_sq, const float *g, int M,
                                     int64_t d, int64_t ld, float lr, float beta1, float beta2, float eps,
                                     float weight_decay, int step, float alpha, float lambda,
                                     float *norms_out, void *ws, size_t ws_bytes, int path,
                                     void *cuda_stream);

/*
 * Round on replicas that live in HOST memory (the arrangement the paper's
 * limitations section mentions: parameters kept off the accelerator).  Copies
 * x_host[M, ld] into the caller's device staging buffer x_dev[M, ld], runs
 * dppf_consensus there, copies the updated replicas back into x_host and, if
 * norms_host != NULL, the M pre-update distances into norms_host (host fp32[M]).
 * All copies are cudaMemcpyAsync on `cuda_stream`; pinned host memory makes them
 * truly asynchronous.  The results are valid once the stream has been
 * synchronised.  x_host needs no particular alignment; x_dev follows the device
 * layout rules.  norms staging uses the workspace.
 */
int dppf_consensus_host(float *x_host, int M, int64_t d, int64_t ld, float alpha, float lambda,
                        float *norms_host, float *x_dev, void *ws, size_t ws_bytes,
                        void *cuda_stream);

/*
 * dppf_consensus with built-in scratch: for callers that cannot allocate.
 * (The paper has no counterpart; this is a convenience of this library.)
 *
 * Some code that wants a round has no way to obtain a workspace: a plugin or callback that
 * is handed device pointers by a host framework and must not allocate behind that
 * framework's memory pool; a training process whose device memory was budgeted and handed
 * out in full at start-up; a latency-critical loop in which allocation calls are banned
 * because they can synchronise the device.  For those callers the per-block partial sums go
 * to a fixed array inside the library's own device memory instead of a caller buffer.
 *
 *  - Same arguments, layout rules, result and return codes as dppf_consensus, minus ws and
 *    ws_bytes.  The call makes no cudaMalloc/cudaFree and uses no allocating library routine.
 *  - Limit: M <= DPPF_STATIC_MAX_WORKERS (16).  A larger M returns DPPF_ERR_WORKSPACE and
 *    nothing is launched.  d is not limited.  The array is 262,656 bytes and every GPU
 *    that loads the library keeps it until the process exits.
 *  - The first call on each device looks up the array's device address (one
 *    cudaGetSymbolAddress with that device current) and remembers it; make that first call
 *    outside any stream capture.
 *  - All calls on a device share the one array, and it keeps whatever the previous call
 *    left.  Nothing in it has to start at zero: every word a round reads it has written
 *    earlier in the same round.  Two calls whose kernels can overlap on the GPU (different
 *    streams without ordering) race on it; order them on one stream or with events.
 */
#define DPPF_STATIC_MAX_WORKERS 16
int dppf_consensus_static(float *x, int M, int64_t d, int64_t ld, float alpha, float lambda,
                          float *norms_out, void *cuda_stream);
/* dppf_device_status for the built-in scratch of the current device: a caller of
 * dppf_consensus_static has no workspace pointer to pass.  Synchronises `cuda_stream`. */
int dppf_static_device_status(void *cuda_stream);

/*
 * Host-side scalars of a DPPF run (no device work, no CUDA call).
 *
 * dppf_lambda_schedule: push strength at iteration t of T (appendix, "How to schedule the
 *   pushing force?"): FIXED lambda; DECREASING lambda/2 (1 + cos(t pi / T)) (follows the
 *   cosine-annealed learning rate); INCREASING lambda/2 (1 - cos(t pi / T)) (the schedule
 *   the paper adopts).  NaN for an unknown kind, T <= 0 or t < 0.
 * dppf_lr_cosine: cosine annealing lr_max/2 (1 + cos(t pi / T)).
 * dppf_qsr_period: communication period of the quadratic synchronisation rule the paper
 *   compares with ("Comparison with Other Communication-Efficient Methods"): max(tau_base, floor((beta / lr_t)^2)); -1 on bad arguments.
 * dppf_round_metrics: from the M pre-round distances r_m (HOST fp32[M], as written to
 *   norms_out and copied back): their mean (the relaxed Mean Valley measure the ablation
 *   plots), the pull strength alpha * r_m per worker (host fp32[M] or NULL) and the push
 *   strength lambda (the push is unit-normed), the two forces whose balance the ablation of
 *   the pull-push mechanism tracks.  Output pointers may be NULL.
 */
#define DPPF_SCHEDULE_FIXED 0
#define DPPF_SCHEDULE_DECREASING 1
#define DPPF_SCHEDULE_INCREASING 2
float dppf_lambda_schedule(int kind, float lambda, int64_t t, int64_t T);
float dppf_lr_cosine(float lr_max, int64_t t, int64_t T);
int64_t dppf_qsr_period(int64_t tau_base, float beta, float lr_t);
int dppf_round_metrics(const float *norms_host, int M, float alpha, float lambda, float *mean_distance,
                       float *pull_strength, float *push_strength);

/*
 * Synchronises `cuda_stream` and returns the status word the kernels keep in the
 * workspace header: DPPF_OK; DPPF_ERR_WORKSPACE if the update pass found a
 * header that its distance pass did not write (workspace overwritten between the
 * two), in which case x was left unchanged; DPPF_ERR_TIMEOUT if a bounded wait on an
 * asynchronous copy gave up (x unchanged if that happened in the distance pass, partly
 * updated otherwise).  DPPF_ERR_CUDA if the stream failed.
 */
int dppf_device_status(const void *ws, void *cuda_stream);

/*
 * Testing hook (the paper has no counterpart).  The kernels that stage rows through shared
 * memory wait for their asynchronous copies with a bounded number of polls (default 2^22,
 * about a second) and report DPPF_ERR_TIMEOUT through the status word if a wait runs out.
 * This sets the poll budget of later calls in this process: first_pass_polls for waits of the
 * distance pass, later_pass_polls for waits of update passes; a negative value restores the
 * default.  A budget of 0 makes every such wait give up at once while the copies themselves
 * still complete (the block waits for them with the full budget before it leaves), which is
 * how the tests drive the give-up path on a healthy GPU.  Applies to dppf_consensus_rounds,
 * dppf_consensus and dppf_consensus_static (staged schedule) and dppf_consensus_general.
 * Always returns DPPF_OK.
 */
int dppf_debug_set_poll_limits(int first_pass_polls, int later_pass_polls);

/*
 * Synchronises `cuda_stream` and returns which schedule the last call on this workspace
 * actually ran (DPPF_PATH_TWO_KERNEL, DPPF_PATH_COOPERATIVE or DPPF_PATH_STAGED): AUTO resolved,
 * and a fallback taken when the runtime refused a cooperative launch made visible.  Two calls
 * on the same input give the same bits if they report the same schedule.  Negative if the
 * stream failed.
 */
int dppf_device_schedule(const void *ws, void *cuda_stream);

/* Static, human-readable name of a dppf_status. */
const char *dppf_status_string(int status);

/* Number of kernel launches the given call shape issues (for launch accounting):
 * fused == 0 dppf_consensus_ex, 1 dppf_local_step_and_consensus_ex, 2 dppf_adamw_step_and_consensus_ex. */
int dppf_launch_count(int M, int64_t d, int path, int fused);

#ifdef __cplusplus
}
#endif
#endif /* DPPF_H */
