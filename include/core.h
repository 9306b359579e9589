/*
 * core.h -- C ABI of the B200 (sm_100a) CORE library.
 *
 * CORE (Common Random Reconstruction) compresses a d-dimensional vector to m
 * scalars by projecting it on m common Gaussian vectors and rebuilds an
 * unbiased estimate from the scalars by regenerating the same vectors
 * (Algorithm 1 of the paper).  With n machines the estimate of the mean
 * gradient is  gtilde = 1/(n m) sum_i sum_j <g_i, xi_j> xi_j  (Section 4,
 * definition of the estimator used by Algorithm 2).
 *
 * Common random vectors (the paper asks only for "a common random number
 * generator"; this is the generator this library fixes):
 *   words   Philox4x32-10, key = (seed mod 2^32, seed >> 32),
 *           counter = (q mod 2^32, q >> 32, j, t); q = k >> 2 is the block of
 *           four coordinates, j the 0-based vector index, t the round.
 *   uniform u(w) = ((w >> 9) + 1/2) 2^-23.
 *   normal  Box-Muller on (w0,w1) and (w2,w3): r = sqrt(-2 ln u(w_even)),
 *           theta = 2 pi u(w_odd); xi_j[4q..4q+3] = (r_a cos th_a, r_a sin th_a,
 *           r_b cos th_b, r_b sin th_b).
 * The vectors are never stored: every kernel regenerates what it needs.
 *
 * Conventions for every entry point
 *   - Pointers named *_dev are DEVICE pointers owned by the caller; *_host are
 *     HOST pointers owned by the caller.  The context owns only its workspace.
 *   - Work is enqueued on the context's stream (core_set_stream; default: the
 *     legacy default stream) and the call returns without synchronising,
 *     except the *_host entry points, which return after their last copy has
 *     completed (also when they fail half-way: no copy is still reading or
 *     writing the caller's buffers after the return), and any call that has to
 *     grow the workspace: core_project, core_round, core_round_host and the
 *     least-squares steps free and re-allocate it (cudaFree / cudaMalloc, which
 *     synchronise the device) when the one they hold is too small.  A caller
 *     that must not meet that synchronisation later takes it up front with
 *     core_reserve_workspace.
 *   - Return value: CORE_OK or a negative error code.  A failing call launches
 *     nothing for CORE_EINVAL; outputs are unspecified after any error, but no
 *     call writes outside the extents stated here.  Nothing prints or aborts.
 *   - One context may be used by one host thread at a time.
 */
#ifndef CORE_B200_CORE_H
#define CORE_B200_CORE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct core_ctx core_ctx;
typedef struct core_ls core_ls;

enum {
    CORE_OK = 0,
    CORE_EINVAL = -1, /* null pointer, non-positive size, ld < d, unknown dtype */
    CORE_ENOMEM = -2, /* workspace allocation failed */
    CORE_ECUDA = -3,  /* CUDA runtime error; code via core_last_cuda_error */
    CORE_ELIMIT = -4  /* size beyond the fixed capacity of an allocation-free entry point */
};

enum { CORE_F32 = 0, CORE_BF16 = 1 };

/* ---- context ------------------------------------------------------------- */

/*
 * Create a context for vectors of dimension d >= 1 compressed to m >= 1 scalars
 * with the common generator keyed by seed.  Round counter starts at t = 0.
 * The ten Philox round keys are derived here, once.  Binds to the CUDA device
 * current at the time of the call.
 */
int core_init(core_ctx **out, uint64_t seed, int64_t d, int32_t m);
int core_destroy(core_ctx *ctx);

/* cuda_stream is a cudaStream_t passed as an opaque pointer (NULL: default stream). */
int core_set_stream(core_ctx *ctx, void *cuda_stream);

/*
 * Round index t selects which "fresh" set xi_1..xi_m is generated (Algorithm 1,
 * first step; Algorithm 2, first step of the loop).  Projection and
 * reconstruction of one communication round must use the same t.
 */
int core_set_round(core_ctx *ctx, uint32_t t);
uint32_t core_get_round(const core_ctx *ctx);

/* Bytes of device workspace the context currently holds. */
size_t core_workspace_bytes(const core_ctx *ctx);

/*
 * Grow the workspace now to what core_project and core_round need for n machines of the given
 * dtype (the context's d and m), so that those calls find it large enough and neither allocate
 * nor synchronise.  May synchronise the device itself.  CORE_ENOMEM leaves the context usable
 * (with no workspace; the next call tries again).
 */
int core_reserve_workspace(core_ctx *ctx, int32_t n, int dtype);

const char *core_strerror(int code);
int core_last_cuda_error(const core_ctx *ctx);

/*
 * Device-side status.  The tensor-memory projection kernel hands buffers between
 * its warps with barriers whose waits are bounded; a wait that runs out makes
 * the kernel finish early (its output is then meaningless) and records a
 * non-zero code in a per-device status word.  A wait gives up after 100 ms of
 * the device's global timer; waits that are served take microseconds.  This call synchronises the
 * current device, stores the word in *status_out (host pointer; 0 = every wait
 * was served) and clears it.  Not part of the paper: run-time diagnostics.
 */
int core_device_status(int32_t *status_out);

/* ---- the round ------------------------------------------------------------- */

/*
 * Projection: P[i*m + j] = <g_i, xi_j>, i < n, j < m (Algorithm 1, sender's
 * step; Algorithm 2, "machine i sends p_ij").
 *   G_dev   n rows of d elements, row i at element offset i*ldg (ldg >= d),
 *           dtype CORE_F32 (float) or CORE_BF16 (bfloat16, widened exactly).
 *           Rows whose byte address and stride are multiples of 16 take the
 *           asynchronous-copy path; any other alignment is handled by an
 *           element-wise path with the same result.
 *   P_dev   n*m floats, row-major.
 * fp32 multiply-add with two-level fp32 accumulation and a fixed reduction
 * order: results are bitwise reproducible for a given (n, m, d, dtype).
 * Machines are processed in groups: up to 64 per pass where the tensor-memory
 * kernel applies (9 or more machines, m >= 96; more than 32 only when m lets a CTA
 * hold 256 vectors, about m >= 256), otherwise up to 16.  The
 * tensor-core kernels form their products with every operand split into a tf32
 * head and tail (same error bar, same reproducibility).  May grow the
 * workspace.
 */
int core_project(core_ctx *ctx, const void *G_dev, int dtype, int32_t n, int64_t ldg, float *P_dev);

/*
 * Aggregation at the central machine (Algorithm 2, "the central machine sends
 * the combined p_ij back"), in the mean convention of the Section-4 estimator
 * (prefactor 1/(n m)):  pbar[j] = (1/n) sum_i P[i*m + j], i ascending.
 */
int core_aggregate(core_ctx *ctx, const float *P_dev, int32_t n, float *pbar_dev);

/*
 * Reconstruction: gtilde[k] = (1/m) sum_j pbar[j] xi_j[k], k < d (Algorithm 1,
 * receiver's step; the equation following Algorithm 1).  gtilde_dev: d floats,
 * each written exactly once.
 */
int core_reconstruct(core_ctx *ctx, const float *pbar_dev, float *gtilde_dev);

/*
 * One whole communication round (Algorithm 2, steps 1-4): project, aggregate,
 * reconstruct with the current t, then t <- t + 1.  pbar_dev (m floats) receives
 * the aggregated message; gtilde_dev (d floats) the estimate.
 */
int core_round(core_ctx *ctx, const void *G_dev, int dtype, int32_t n, int64_t ldg, float *pbar_dev,
               float *gtilde_dev);

/*
 * The same round with HOST buffers: G_host (n rows, stride ldg elements) is
 * streamed to the device in coordinate slabs that are projected as they
 * arrive; gtilde_host (d floats) and pbar_host (m floats) are copied back, the
 * reconstruction being produced and copied slab by slab.  Pinned host memory
 * gives asynchronous copies; pageable memory works but serialises.  Returns
 * after the last copy has completed.  t <- t + 1.
 */
int core_round_host(core_ctx *ctx, const void *G_host, int dtype, int32_t n, int64_t ldg,
                    float *pbar_host, float *gtilde_host);

/*
 * Projection without any device allocation (the paper has no counterpart: this entry point
 * exists for the library's users, not for the method).
 *
 * Who needs it: callers that cannot call cudaMalloc -- an application whose memory pool has
 * claimed the whole device, or code on a path where the allocator's implicit device-wide
 * synchronisation is not allowed.  core_init and core_project obtain a workspace with
 * cudaMalloc; this call takes no context and obtains nothing.  The per-CTA partial sums of
 * the projection go to a fixed array of CORE_STATIC_SCRATCH_FLOATS floats (4 MiB) that is
 * part of the library image: every GPU onto which the library's code has been loaded holds it
 * until the process exits.
 *
 * Computes P[i*m + j] = <g_i, xi_j> exactly as core_project does for the generator keyed by
 * (seed, round t); arguments as for core_project, plus d, m, seed and t passed directly.
 * cuda_stream: the stream to enqueue on (NULL: default stream); returns without
 * synchronising.  cuda_error_out (may be NULL) receives the CUDA error code when the return
 * value is CORE_ECUDA.
 *
 * Limits: n <= 16 and n*m <= CORE_STATIC_SCRATCH_FLOATS, otherwise CORE_ELIMIT and nothing is
 * launched.  When the usual number of CTA columns does not fit the array, fewer columns are
 * used: slower, and the result may differ from core_project's in the last bits (same bound
 * against the exact value).
 *
 * The first call on a device is a set-up call: it looks up the array's device address, and with
 * CUDA's default lazy module loading that is also when the driver loads this part of the library
 * onto the device and reserves the 4 MiB (the kernels are loaded at their first launch likewise).
 * So the first call per device can itself need device memory, and can fail with CORE_ECUDA on a
 * device that is already full: make it early, before the application claims the device, and
 * outside any stream capture.  Later calls allocate nothing.  (With CUDA_MODULE_LOADING=EAGER in
 * the environment the cost moves to the moment the library is loaded.)
 * G_dev and P_dev must belong to the current device (checked; CORE_EINVAL otherwise): the scratch
 * array used is the current device's.
 * All calls share the one array, which keeps the previous call's contents: nothing in it
 * needs to start at zero (every entry is written before it is read within a call), but two
 * calls whose kernels overlap on the GPU -- different streams, no dependency between them --
 * race on it.  Calls on one stream, or ordered by events, are safe.
 */
#define CORE_STATIC_SCRATCH_FLOATS ((size_t)1 << 20)
int core_project_static(uint64_t seed, uint32_t t, int64_t d, int32_t m, const void *G_dev, int dtype,
                        int32_t n, int64_t ldg, float *P_dev, void *cuda_stream, int *cuda_error_out);

/* ---- least-squares CORE-GD driver (Algorithm 2) ----------------------------- */

/*
 * f(x) = (1/n) sum_i 1/(2 rows) ||A_i x - b_i||^2 : the ridge-separable form of
 * Section 4 with quadratic loss and no ridge term.  A_dev is n x rows x d floats
 * row-major, b_dev n x rows floats; both are borrowed (must outlive the handle).
 * The handle owns the gradient matrix G[n x d] and its partial sums.
 */
int core_ls_create(core_ls **out, const float *A_dev, const float *b_dev, int32_t n, int32_t rows,
                   int64_t d);
int core_ls_destroy(core_ls *ls);

/*
 * One iteration of Algorithm 2: g_i = A_i^T (A_i x - b_i) / rows for every
 * machine, one round with the context's current t (then t <- t + 1), and
 * x <- x - h * gtilde.  x_dev: d floats, updated in place.  ctx must have been
 * created with the same d.  The update is applied inside the reconstruction
 * kernel; the estimate itself is not stored.
 */
int core_gd_step(core_ctx *ctx, core_ls *ls, float h, float *x_dev);

/*
 * One iteration of CORE-AGD (the accelerated, heavy-ball variant in the paper's
 * appendix "Acceleration of CORE-GD", Algorithm 4):
 *   y = x + (1 - beta)(x - x_prev);  gtilde = one round on the machine gradients
 *   at y (current t, then t <- t + 1);  x_prev <- x;  x <- y - h * gtilde.
 * The gradient is taken at y, as the algorithm's update line states (its displayed
 * reconstruction formula prints x).  x_dev, x_prev_dev: d floats each, distinct,
 * both updated in place; for the first iteration pass x_prev = x.
 */
int core_agd_step(core_ctx *ctx, core_ls *ls, float h, float beta, float *x_dev, float *x_prev_dev);

/*
 * One iteration of the variant with the comparison step ("CORE-GD in Non-convex
 * Optimization", Algorithm 3) with a step h fixed by the caller (its Option II, where h
 * depends only on constants of the problem): trial point x~ = x - h * gtilde(x) from one
 * round (current t, then t <- t + 1); x <- argmin over {x, x~} of f, a tie keeping x.
 *   f_dev         one double: f(x) on entry, f of the kept point on return
 *   accepted_dev  one int32 (may be NULL): 1 if the trial point was taken
 * The comparison is made on the device; the call does not synchronise.
 */
int core_gd_step_guarded(core_ctx *ctx, core_ls *ls, float h, float *x_dev, double *f_dev,
                         int32_t *accepted_dev);

/*
 * The same iteration with Option I of Algorithm 3: the step is chosen from the size of the combined
 * messages of this very round,
 *     p = sqrt((1/m) sum_j pbar_j^2),   h = min{ m / (16 r1), c H^(-1/2) p^(-1/2) d^(-3/4) m^(3/4) },
 * r1 a bound on the trace of the Hessian, H the Lipschitz constant of the Hessian, c the algorithm's
 * constant (it prints 1/1600); all three > 0.  The algorithm's own line for p has its index ranges
 * swapped and, read literally, is a mean of zero-mean numbers that cannot bound the gradient norm as
 * the proof requires; the root mean square above is the reading taken (its square has expectation
 * ||mean gradient||^2, by the law of the messages).  p and h are formed on the device (in double,
 * stored as float) between aggregation and reconstruction; nothing synchronises.
 *   f_dev, accepted_dev  as for core_gd_step_guarded
 *   p_dev, h_dev         one float each (may be NULL): the statistic and the step of this iteration
 */
int core_gd_step_option1(core_ctx *ctx, core_ls *ls, double r1, double H, double c, float *x_dev, double *f_dev,
                         int32_t *accepted_dev, float *p_dev, float *h_dev);

/* ---- decentralised CORE-GD (appendix "Decentralized CORE Based Algorithms", Algorithm 5) ------- */

/*
 * One gossip round on the machines' messages: P_out[i*m + j] = sum_l W[i*n + l] P_in[l*m + j], l
 * ascending, fp32.  W_dev: the n x n gossip matrix of the network, row-major (symmetric, doubly
 * stochastic, zero between machines that are not neighbours); P_in_dev, P_out_dev: n x m, distinct.
 * Repeated rounds solve the algorithm's m-dimensional averaging problem, whose solution is
 * p = (1/n) sum_i p_i: every row tends to it at the rate of W's second largest eigenvalue modulus.
 */
int core_gossip_round(core_ctx *ctx, const float *W_dev, const float *P_in_dev, int32_t n, float *P_out_dev);

/*
 * One iteration of Algorithm 5 on the least-squares objective, all n machines simulated on this GPU:
 * every machine projects its own gradient (current t), `rounds` gossip rounds with W_dev replace the
 * central machine, machine `reader`'s estimate of p is reconstructed and x <- x - h * estimate (inside
 * the reconstruction), then t <- t + 1.  The algorithm presumes the averaging problem solved to
 * accuracy: spread_dev (one float, may be NULL) receives max_ij |estimate_i[j] - estimate_reader[j]|,
 * which tells whether `rounds` was enough.  as_printed = 0: prefactor 1/m, the mean convention of the
 * Section-4 estimator used everywhere in this library; as_printed != 0: the printed n/m (the same
 * direction, n times as long).
 */
int core_decentralized_step(core_ctx *ctx, core_ls *ls, const float *W_dev, int32_t rounds, int32_t reader,
                            int as_printed, float h, float *x_dev, float *spread_dev);

/*
 * f(x) as a double, computed on the device in a fixed order (the objective of Algorithm 2's
 * least-squares instance).  core_ls_loss leaves it in loss_dev[0] (DEVICE pointer: the guarded step
 * consumes it there without a host round trip); core_ls_loss_host also enqueues its copy to
 * loss_host[0] (HOST pointer, pinned for an asynchronous copy) on the context's stream: read it
 * after synchronising that stream.  Neither call synchronises.
 */
int core_ls_loss(core_ctx *ctx, core_ls *ls, const float *x_dev, double *loss_dev);
int core_ls_loss_host(core_ctx *ctx, core_ls *ls, const float *x_dev, double *loss_host);

/* G_out_dev[i*d + k] = g_i[k] at x (the machine gradients alone; n*d floats). */
int core_ls_gradients(core_ctx *ctx, core_ls *ls, const float *x_dev, float *G_out_dev);

/* ---- failure paths, made on the host or bounded on the device (no counterpart in the paper) ---- */

/*
 * Which projection kernel later calls use: -1 the library's choice by shape (default), 0 the scalar
 * kernel, 1 the warp-level tensor-core kernel where its shape limits allow, 2 the tensor-memory
 * (tcgen05) kernel for every group of machines it can take (up to 64).  Process-wide; for measuring where one kernel
 * overtakes the other and for testing each on shapes the default would not give it.
 */
int core_debug_force_project_kernel(int kind);

/*
 * The next `count` device allocations of this library fail as if the device were out of memory
 * (count = 0 switches this off).  Lets a test see CORE_ENOMEM from core_init, core_project,
 * core_round_host, core_ls_create ... without exhausting a GPU: a failing call launches nothing and
 * leaves its context usable.
 */
int core_debug_fail_allocations(int count);

/*
 * Runs one small CTA whose first warp waits, with the bounded-wait helper of the tensor-memory
 * projection, on a barrier that nobody completes; after limit_us microseconds (1..100000) the wait
 * gives up, the device status word receives `code` (>= 1; read and clear it with
 * core_device_status) and the kernel returns by its normal exit.  observed_host[0] = 0 if the wait
 * ran out (1 if it was served, which cannot happen), observed_host[1] = 1 if the CTA's second warp
 * saw the abort flag.  Synchronises.  Uses no tensor-core instruction.
 */
int core_debug_wait_timeout(uint32_t limit_us, int32_t code, uint32_t observed_host[2]);

/* ---- generator windows (for checking the generator itself) ------------------- */

/* words_dev[4*(q-q0) + l] = word l of block q of vector j, q0 <= q < q0+nq, current t. */
int core_debug_philox(core_ctx *ctx, uint32_t j, uint64_t q0, int64_t nq, uint32_t *words_dev);
/* z_dev[4*(q-q0) + l] = xi_j[4q + l]. */
int core_debug_gaussians(core_ctx *ctx, uint32_t j, uint64_t q0, int64_t nq, float *z_dev);
/* Box-Muller alone: z_dev[4b..4b+3] from the caller's words_dev[4b..4b+3], b < nb. */
int core_debug_box_muller(core_ctx *ctx, const uint32_t *words_dev, int64_t nb, float *z_dev);

/*
 * Launch geometry the projection would use for the first pass over n machines (at most 64 per pass),
 * m vectors and d coordinates on a device with sm_count SMs.  Host-only: touches no device.
 * out[0..9] = machines per pass (rounded up to a power of two; 16, 32 or 64 for the tensor-memory kernel), vectors per thread,
 * coordinate blocks per thread step, blocks per shared-memory tile, threads across
 * vectors, threads across blocks, CTAs across coordinates, CTAs across vectors,
 * tiles of d, dynamic shared memory bytes.
 */
int core_debug_project_plan(int32_t n, int32_t m, int64_t d, int dtype, int32_t sm_count, int64_t out[10]);

/*
 * Instruction-rate probes (no counterpart in the paper: they support the roofline of the round kernels,
 * which are bound by instruction issue).  Kind k < core_debug_pipe_kinds() - 3 runs a loop whose body
 * is counts_out[0..6] = (32x32-bit multiplies keeping the high word, fp32 multiply-adds, packed fp32 multiply-adds,
 * three-input logic ops, special-function calls, fp64 multiply-adds, 32-bit integer multiply-adds),
 * all on independent chains (core_debug_pipe_mix reports the counts, all zero for the last three
 * kinds).  The last three kinds run rounds 2..9 of Philox for four counters per body with the wide
 * multiply done by the integer multiplier, by the fp64 unit plus a 32-bit multiply, or half and half;
 * their checksums must agree (same words).
 * core_debug_pipe_cycles launches the loop on every SM with warps_per_scheduler (2, 4 or 8) warps
 * resident per scheduler, synchronises, and stores in *cycles_per_body_out (host pointer) the SM cycles
 * one scheduler spends per loop body and warp, and in *checksum_out (host pointer, may be NULL) a
 * digest of the loop results.  Allocates and frees its own small device buffers.
 */
int core_debug_pipe_kinds(void);
int core_debug_pipe_mix(int kind, int32_t counts_out[7]);
int core_debug_pipe_cycles(int kind, int warps_per_scheduler, int iters, uint32_t seed, double *cycles_per_body_out,
                           uint32_t *checksum_out);

#ifdef __cplusplus
}
#endif
#endif
