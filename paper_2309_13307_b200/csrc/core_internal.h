// Internal declarations shared by the translation units of the CORE library.
#pragma once

#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

#include "core_rng.cuh"

namespace core {

constexpr int kThreads = 256;        // threads per CTA in the round kernels
constexpr int kMaxGroup = 16;        // machines handled by one pass of the scalar projection
constexpr int kMaxGroupTc = 64;      // most machines one pass of the tensor-memory projection can take

// Machines the next projection pass takes when n_left remain: up to 64 (32 where a CTA holds one group of
// 128 vectors only) where the tensor-memory kernel applies to more than 16, otherwise at most 16.
int32_t project_group(int32_t n_left, int32_t m);
// Test hook: -1 = choose by shape (default); 0 = always the scalar kernel; 1 = the warp-level tensor-core
// kernel where its shape limits allow; 2 = the tensor-memory kernel for any group of machines it can take.
void project_force_kernel(int kind);

// Launch geometry of one projection pass, fixed by (n, m, d, dtype) on the host.
struct ProjectPlan {
    int nb;           // machines per pass rounded up to 1, 2, 4, 8 or 16
    int jt;           // vectors per thread
    int uq;           // coordinate blocks per thread per step
    int tile_q;       // coordinate blocks (of 4) per shared-memory tile
    int tj;           // threads across vectors (power of two)
    int tq;           // threads across coordinate blocks = kThreads / tj
    int grid_x;       // CTAs across coordinates
    int grid_y;       // CTAs across vectors
    int64_t tiles;    // ceil(d / (4 * tile_q))
    size_t smem;      // dynamic shared memory per CTA
    int mma;          // 0: scalar kernel; 1: warp-level tensor-core kernel; 2: tcgen05 kernel
};

ProjectPlan make_project_plan(int32_t n_group, int32_t m, int64_t d, int dtype, int sm_count);

// Tensor-core variant of the projection pass (core_project_mma.cu); same partial-sum layout.
bool project_mma_applies(int32_t n_group, int32_t m);
void fill_project_mma_plan(ProjectPlan &plan, int32_t m, int64_t d, int dtype, int sm_count);
cudaError_t launch_project_mma(const ProjectPlan &plan, const RoundKeys &keys, uint32_t t, const void *G,
                               int dtype, int32_t n, int64_t ldg, int64_t d, int32_t m, uint64_t q_base,
                               float *partial, cudaStream_t stream);

// tcgen05 variant (core_project_tc.cu): 128 or 256 vectors per CTA, up to project_tc_max_group(m) machines per
// pass (N = 16, 32 or 64 of the instruction), accumulators in tensor memory; same partial-sum layout.  q_base must be a multiple of 64 blocks.  Its waits are bounded: a wait that
// runs out raises a device status word, which project_tc_take_status returns and clears after
// synchronising the device.
bool project_tc_applies(int32_t n_group, int32_t m);
int32_t project_tc_max_group(int32_t m);   // 64 with 256 vectors per CTA, otherwise 32
void fill_project_tc_plan(ProjectPlan &plan, int32_t n_group, int32_t m, int64_t d, int dtype, int sm_count);
cudaError_t launch_project_tc(const ProjectPlan &plan, const RoundKeys &keys, uint32_t t, const void *G,
                              int dtype, int32_t n, int64_t ldg, int64_t d, int32_t m, uint64_t q_base,
                              float *partial, cudaStream_t stream);
cudaError_t project_tc_take_status(int *status);
// One small CTA that waits, with the projection's bounded-wait helper, on a barrier nobody completes:
// after limit_ns the wait gives up, the status word receives `code`, and observed_dev[0..1] (device)
// become {0: the wait did not succeed, 1: the second warp saw the abort flag}.
cudaError_t launch_wait_timeout_probe(uint64_t limit_ns, int code, uint32_t *observed_dev, cudaStream_t stream);

// One projection pass over coordinates [0, d) of rows G + i*ldg, i < n <= 16.
// q_base is the global index of the block holding coordinate 0 of G (non-zero when G
// is a slab of a longer vector).  Writes partial[(c * n + i) * m + j], c < plan.grid_x.
// With splits > 0 (fp32, scalar kernel only: plan.mma == 0) row i is not stored anywhere: it is
// scale * (G[(i*splits + 0)*ldg + k] + ... + G[(i*splits + splits-1)*ldg + k]), summed in that order
// while the tile is staged (the per-row-range partial gradients of the least-squares kernels).
cudaError_t launch_project(const ProjectPlan &plan, const RoundKeys &keys, uint32_t t, const void *G,
                           int dtype, int32_t n, int64_t ldg, int64_t d, int32_t m, uint64_t q_base,
                           float *partial, cudaStream_t stream, int splits = 0, float scale = 1.0f);

// P[i*m+j] = (accumulate ? P[i*m+j] : 0) + sum_c partial[c][i][j], c ascending.
cudaError_t launch_finish_project(const float *partial, int chunks, int32_t n, int32_t m, float *P,
                                  bool accumulate, cudaStream_t stream);

// pbar[j] = (1/n) sum_i (sum_c partial[c][i][j]): finish + aggregate for one group of machines, same order.
cudaError_t launch_finish_aggregate(const float *partial, int chunks, int32_t n, int32_t m, float *pbar,
                                    cudaStream_t stream);

cudaError_t launch_aggregate(const float *P, int32_t n, int32_t m, float *pbar, cudaStream_t stream);

// out[k - k_begin] = gtilde[k] for k in [k_begin, k_end); k_begin must be a multiple of 2048.
// With an epilogue the estimate is consumed where it is produced and never stored:
//   out[k] = base[k] - step * gtilde[k]   (the optimiser update of Algorithms 2 and 4)
// and, if shift_dst is set, shift_dst[k] = shift_src[k] first (x_prev <- x of Algorithm 4).
// out may alias base and shift_src; all four arrays are indexed like out.
// step_dev, when set, overrides step: the kernel reads the step from device memory (a step that an
// earlier kernel of the same iteration chose, as in Option I of Algorithm 3), times step_scale.
struct ReconstructEpilogue {
    const float *base;
    float step;
    const float *shift_src;
    float *shift_dst;
    const float *step_dev = nullptr;
    float step_scale = 1.0f;
};
cudaError_t launch_reconstruct(const RoundKeys &keys, uint32_t t, const float *pbar, int32_t m,
                               int64_t k_begin, int64_t k_end, float *out, int sm_count,
                               cudaStream_t stream, const ReconstructEpilogue *epilogue = nullptr);

// y[k] = x[k] + gamma * (x[k] - x_prev[k])   (look-ahead point of Algorithm 4)
cudaError_t launch_lookahead(const float *x, const float *x_prev, float gamma, int64_t d, float *y,
                             cudaStream_t stream);

cudaError_t launch_debug_philox(const RoundKeys &keys, uint32_t t, uint32_t j, uint64_t q0, int64_t nq,
                                uint32_t *words, cudaStream_t stream);
cudaError_t launch_debug_gaussians(const RoundKeys &keys, uint32_t t, uint32_t j, uint64_t q0, int64_t nq,
                                   float *z, cudaStream_t stream);
cudaError_t launch_debug_box_muller(const uint32_t *words, int64_t nb, float *z, cudaStream_t stream);

// Least squares.  Pass 1: res[i*rows + r] = A_i[r] . x - b_i[r].  Pass 2: the rows of a
// machine are cut into `splits` ranges; part[(i*splits + s)*d + k] = sum over the rows of
// range s of A_i[r][k] * res_i[r].  Reduce: G[i*d + k] = (1/rows) sum_s part[i][s][k].
struct LsPlan {
    int splits;
    int rows_per_split;
};
LsPlan make_ls_plan(int32_t n, int32_t rows, int64_t d, int sm_count);
cudaError_t launch_ls_residual(const float *A, const float *b, const float *x, int32_t n, int32_t rows,
                               int64_t d, float *res, cudaStream_t stream);
cudaError_t launch_ls_at_r(const LsPlan &plan, const float *A, const float *res, int32_t n, int32_t rows,
                           int64_t d, float *part, cudaStream_t stream);
cudaError_t launch_ls_reduce(const LsPlan &plan, const float *part, int32_t n, int32_t rows, int64_t d,
                             float *G, cudaStream_t stream);
// Single pass over A for d <= 8192, d % 4 == 0: part[(i*splits + s)*d + k] as above, with the
// residual of each row formed on the fly (A is read from HBM once instead of twice).  A plan with
// splits == 0 means the single-pass kernel does not apply to this shape.
LsPlan make_ls_fused_plan(int32_t n, int32_t rows, int64_t d, int sm_count);
bool ls_fused_usable(const LsPlan &fused_plan, const float *A, const float *x, const float *part);
cudaError_t launch_ls_fused(const LsPlan &plan, const float *A, const float *b, const float *x, int32_t n,
                            int32_t rows, int64_t d, float *part, cudaStream_t stream);
// Comparison step of Algorithm 3, on the device: if *f_trial < *f then x <- trial, *f <- *f_trial and the
// flag is 1, otherwise nothing changes and the flag is 0 (a tie keeps x).  flag_scratch is a device int
// owned by the caller of this function; flag_out (may be null) receives a copy.
cudaError_t launch_keep_better(const double *f_trial, const float *trial, int64_t d, double *f, float *x,
                               int *flag_scratch, int32_t *flag_out, cudaStream_t stream);
// loss[0] = (1/n) sum_i 1/(2 rows) sum_r res_i[r]^2, summed in double in a fixed order
cudaError_t launch_ls_loss(const float *res, int32_t n, int32_t rows, double *loss, cudaStream_t stream);

// Option I of Algorithm 3: p_out[0] (may be null) = sqrt((1/m) sum_j pbar_j^2), h_out[0] =
// min{ m / (16 r1), c H^-1/2 p^-1/2 d^-3/4 m^3/4 }, both formed on the device in double and stored as float.
cudaError_t launch_option1_step(const float *pbar, int32_t m, int64_t d, double r1, double H, double c, float *p_out,
                                float *h_out, cudaStream_t stream);
// Algorithm 5's averaging by gossip: out[i*m + j] = sum_l W[i*n + l] in[l*m + j], l ascending (in != out).
cudaError_t launch_gossip_round(const float *W, const float *in, int32_t n, int32_t m, float *out, cudaStream_t stream);
// spread[0] = max_ij |P[i*m + j] - P[reader*m + j]|
cudaError_t launch_consensus_spread(const float *P, int32_t n, int32_t m, int32_t reader, float *spread,
                                    cudaStream_t stream);

}  // namespace core
