// C ABI of the CORE library: argument checks, context, workspace and stream plumbing.
// Every entry point is declared, with its contract, in include/core.h.
#include "core.h"

#include <atomic>
#include <new>

#include "core_internal.h"

using namespace core;

struct core_ctx {
    uint64_t seed;
    int64_t d;
    int32_t m;
    uint32_t t;
    int device;
    int sm_count;
    cudaStream_t stream;
    RoundKeys keys;
    void *ws;            // device workspace, grown on demand
    size_t ws_bytes;
    float *pbar;         // m floats, for callers that do not keep the message (gd step)
    int last_cuda;
    // host-streaming state (core_round_host), created on first use
    cudaStream_t copy_stream, work_stream;
    cudaEvent_t in_ready[2], in_free[2], out_ready[2], out_free[2];
    bool host_ready;
    void *slab;          // 2 input slabs + 2 output slabs
    size_t slab_bytes;
};

struct core_ls {
    const float *A;
    const float *b;
    int32_t n, rows;
    int64_t d;
    int device;
    LsPlan plan;         // two passes over A (any shape)
    LsPlan fused_plan;   // one pass over A (d <= 8192, d % 4 == 0); splits == 0 if it does not apply
    float *res;          // n*rows
    float *part;         // n*splits*d
    float *G;            // n*d
    float *y;            // d: look-ahead point of the accelerated step / trial point of the guarded step
    double *f_trial;     // loss at the trial point
    int *accepted;       // 1 if the last guarded step took the trial point
    float *step;         // step chosen on the device (Option I of Algorithm 3), then its statistic p
};

namespace {

size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int cuda_fail(core_ctx *ctx, cudaError_t e) {
    if (ctx) ctx->last_cuda = (int)e;
    return e == cudaErrorMemoryAllocation ? CORE_ENOMEM : CORE_ECUDA;
}

#define CORE_CUDA(ctx, expr)                                  \
    do {                                                      \
        cudaError_t e__ = (expr);                             \
        if (e__ != cudaSuccess) return cuda_fail((ctx), e__); \
    } while (0)

// Every device allocation of the library goes through here, so that tests can make the next ones fail
// on the host (core_debug_fail_allocations) and see the out-of-memory paths without exhausting a GPU.
std::atomic<int> g_fail_allocations{0};

cudaError_t core_malloc(void **out, size_t bytes) {
    int left = g_fail_allocations.load();
    while (left > 0) {
        if (g_fail_allocations.compare_exchange_weak(left, left - 1)) {
            *out = nullptr;
            return cudaErrorMemoryAllocation;
        }
    }
    return cudaMalloc(out, bytes);
}

bool on_device(int device) {
    int cur = -1;
    return cudaGetDevice(&cur) == cudaSuccess && cur == device;
}

int ensure_workspace(core_ctx *ctx, size_t bytes) {
    if (bytes <= ctx->ws_bytes) return CORE_OK;
    if (ctx->ws) {
        cudaError_t e = cudaFree(ctx->ws);   // waits for work that may still use it
        ctx->ws = nullptr;
        ctx->ws_bytes = 0;
        if (e != cudaSuccess) return cuda_fail(ctx, e);
    }
    bytes = round_up(bytes, (size_t)1 << 20);
    cudaError_t e = core_malloc(&ctx->ws, bytes);
    if (e != cudaSuccess) {
        ctx->ws = nullptr;
        cudaGetLastError();
        ctx->last_cuda = (int)e;
        return CORE_ENOMEM;
    }
    ctx->ws_bytes = bytes;
    return CORE_OK;
}

bool valid_dtype(int dtype) { return dtype == CORE_F32 || dtype == CORE_BF16; }
size_t elem_size(int dtype) { return dtype == CORE_BF16 ? 2 : 4; }

// Bytes of partial sums the projection of n machines needs (largest group of a pass).
size_t partial_bytes(const core_ctx *ctx, int32_t n, int64_t d, int dtype) {
    size_t need = 0;
    for (int32_t i0 = 0, ng = 0; i0 < n; i0 += ng) {
        ng = project_group(n - i0, ctx->m);
        const ProjectPlan plan = make_project_plan(ng, ctx->m, d, dtype, ctx->sm_count);
        const size_t b = (size_t)plan.grid_x * ng * ctx->m * sizeof(float);
        if (b > need) need = b;
    }
    return round_up(need, 256);
}

// Projects rows [0, n) of a matrix whose coordinate 0 is global block q_base; the partial
// sums go through `partial`; P (n*m) receives (or accumulates) the result.
int project_into(core_ctx *ctx, const void *G, int dtype, int32_t n, int64_t ldg, int64_t d, uint64_t q_base,
                 float *partial, float *P, bool accumulate, cudaStream_t stream) {
    for (int32_t i0 = 0, ng = 0; i0 < n; i0 += ng) {
        ng = project_group(n - i0, ctx->m);
        const ProjectPlan plan = make_project_plan(ng, ctx->m, d, dtype, ctx->sm_count);
        const char *rows = static_cast<const char *>(G) + (size_t)i0 * (size_t)ldg * elem_size(dtype);
        CORE_CUDA(ctx, launch_project(plan, ctx->keys, ctx->t, rows, dtype, ng, ldg, d, ctx->m, q_base, partial,
                                      stream));
        CORE_CUDA(ctx, launch_finish_project(partial, plan.grid_x, ng, ctx->m, P + (size_t)i0 * ctx->m, accumulate,
                                             stream));
    }
    return CORE_OK;
}

int check_ctx(const core_ctx *ctx) {
    if (!ctx) return CORE_EINVAL;
    if (!on_device(ctx->device)) return CORE_EINVAL;
    return CORE_OK;
}

}  // namespace

extern "C" {

int core_init(core_ctx **out, uint64_t seed, int64_t d, int32_t m) {
    if (!out) return CORE_EINVAL;
    *out = nullptr;
    if (d < 1 || m < 1) return CORE_EINVAL;
    core_ctx *ctx = new (std::nothrow) core_ctx();
    if (!ctx) return CORE_ENOMEM;
    ctx->seed = seed;
    ctx->d = d;
    ctx->m = m;
    ctx->t = 0;
    ctx->stream = nullptr;
    ctx->keys = expand_keys(seed);
    ctx->ws = nullptr;
    ctx->ws_bytes = 0;
    ctx->pbar = nullptr;
    ctx->last_cuda = 0;
    ctx->host_ready = false;
    ctx->slab = nullptr;
    ctx->slab_bytes = 0;
    cudaError_t e = cudaGetDevice(&ctx->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device);
    if (e == cudaSuccess) e = core_malloc(reinterpret_cast<void **>(&ctx->pbar), (size_t)m * sizeof(float));
    if (e != cudaSuccess) {
        cudaGetLastError();
        const int rc = e == cudaErrorMemoryAllocation ? CORE_ENOMEM : CORE_ECUDA;
        delete ctx;
        return rc;
    }
    *out = ctx;
    return CORE_OK;
}

int core_destroy(core_ctx *ctx) {
    if (!ctx) return CORE_EINVAL;
    int rc = CORE_OK;
    if (ctx->ws && cudaFree(ctx->ws) != cudaSuccess) rc = CORE_ECUDA;
    if (ctx->pbar && cudaFree(ctx->pbar) != cudaSuccess) rc = CORE_ECUDA;
    if (ctx->slab && cudaFree(ctx->slab) != cudaSuccess) rc = CORE_ECUDA;
    if (ctx->host_ready) {
        cudaStreamDestroy(ctx->copy_stream);
        cudaStreamDestroy(ctx->work_stream);
        for (int s = 0; s < 2; ++s) {
            cudaEventDestroy(ctx->in_ready[s]);
            cudaEventDestroy(ctx->in_free[s]);
            cudaEventDestroy(ctx->out_ready[s]);
            cudaEventDestroy(ctx->out_free[s]);
        }
    }
    delete ctx;
    return rc;
}

int core_set_stream(core_ctx *ctx, void *cuda_stream) {
    if (!ctx) return CORE_EINVAL;
    ctx->stream = static_cast<cudaStream_t>(cuda_stream);
    return CORE_OK;
}

int core_set_round(core_ctx *ctx, uint32_t t) {
    if (!ctx) return CORE_EINVAL;
    ctx->t = t;
    return CORE_OK;
}

uint32_t core_get_round(const core_ctx *ctx) { return ctx ? ctx->t : 0u; }

size_t core_workspace_bytes(const core_ctx *ctx) {
    return ctx ? ctx->ws_bytes + ctx->slab_bytes + (size_t)ctx->m * sizeof(float) : 0;
}

const char *core_strerror(int code) {
    switch (code) {
        case CORE_OK: return "ok";
        case CORE_EINVAL: return "invalid argument";
        case CORE_ENOMEM: return "out of device memory";
        case CORE_ECUDA: return "CUDA runtime error";
        case CORE_ELIMIT: return "size exceeds the fixed capacity of this entry point";
        default: return "unknown error";
    }
}

int core_last_cuda_error(const core_ctx *ctx) { return ctx ? ctx->last_cuda : 0; }

int core_device_status(int32_t *status_out) {
    if (!status_out) return CORE_EINVAL;
    int status = 0;
    if (project_tc_take_status(&status) != cudaSuccess) {
        cudaGetLastError();
        return CORE_ECUDA;
    }
    *status_out = status;
    return CORE_OK;
}

int core_project(core_ctx *ctx, const void *G_dev, int dtype, int32_t n, int64_t ldg, float *P_dev) {
    if (int rc = check_ctx(ctx)) return rc;
    if (!G_dev || !P_dev || n < 1 || ldg < ctx->d || !valid_dtype(dtype)) return CORE_EINVAL;
    if (int rc = ensure_workspace(ctx, partial_bytes(ctx, n, ctx->d, dtype))) return rc;
    return project_into(ctx, G_dev, dtype, n, ldg, ctx->d, 0, static_cast<float *>(ctx->ws), P_dev, false,
                        ctx->stream);
}

int core_reserve_workspace(core_ctx *ctx, int32_t n, int dtype) {
    if (int rc = check_ctx(ctx)) return rc;
    if (n < 1 || !valid_dtype(dtype)) return CORE_EINVAL;
    // what core_round needs (partial sums + the messages); core_project needs the first part only
    const size_t pb = partial_bytes(ctx, n, ctx->d, dtype);
    const size_t Pb = round_up((size_t)n * ctx->m * sizeof(float), 256);
    return ensure_workspace(ctx, pb + Pb);
}

int core_aggregate(core_ctx *ctx, const float *P_dev, int32_t n, float *pbar_dev) {
    if (int rc = check_ctx(ctx)) return rc;
    if (!P_dev || !pbar_dev || n < 1) return CORE_EINVAL;
    CORE_CUDA(ctx, launch_aggregate(P_dev, n, ctx->m, pbar_dev, ctx->stream));
    return CORE_OK;
}

int core_reconstruct(core_ctx *ctx, const float *pbar_dev, float *gtilde_dev) {
    if (int rc = check_ctx(ctx)) return rc;
    if (!pbar_dev || !gtilde_dev) return CORE_EINVAL;
    CORE_CUDA(ctx, launch_reconstruct(ctx->keys, ctx->t, pbar_dev, ctx->m, 0, ctx->d, gtilde_dev, ctx->sm_count,
                                      ctx->stream));
    return CORE_OK;
}

// A step chosen on the device from the combined messages, between aggregation and reconstruction
// (Option I of Algorithm 3): h_dev receives the step, p_dev (may be null) the statistic.
struct StepRule {
    double r1, H, c;
    float *p_dev;
    float *h_dev;
};

static int apply_step_rule(core_ctx *ctx, const StepRule *rule, const float *pbar_dev) {
    if (!rule) return CORE_OK;
    CORE_CUDA(ctx, launch_option1_step(pbar_dev, ctx->m, ctx->d, rule->r1, rule->H, rule->c, rule->p_dev, rule->h_dev,
                                       ctx->stream));
    return CORE_OK;
}

// project -> aggregate -> reconstruct with the current t, then t <- t + 1.  With an epilogue the
// reconstruction writes the optimiser update into `out` instead of the estimate.
static int round_with_epilogue(core_ctx *ctx, const void *G_dev, int dtype, int32_t n, int64_t ldg, float *pbar_dev,
                               float *out, const ReconstructEpilogue *epilogue, const StepRule *rule = nullptr) {
    const size_t pb = partial_bytes(ctx, n, ctx->d, dtype);
    const size_t Pb = round_up((size_t)n * ctx->m * sizeof(float), 256);
    if (int rc = ensure_workspace(ctx, pb + Pb)) return rc;
    float *partial = static_cast<float *>(ctx->ws);
    float *P = reinterpret_cast<float *>(static_cast<char *>(ctx->ws) + pb);
    if (project_group(n, ctx->m) == n) {
        // one group of machines: the per-machine messages are not kept, so they are never written
        const ProjectPlan plan = make_project_plan(n, ctx->m, ctx->d, dtype, ctx->sm_count);
        CORE_CUDA(ctx, launch_project(plan, ctx->keys, ctx->t, G_dev, dtype, n, ldg, ctx->d, ctx->m, 0, partial,
                                      ctx->stream));
        CORE_CUDA(ctx, launch_finish_aggregate(partial, plan.grid_x, n, ctx->m, pbar_dev, ctx->stream));
    } else {
        if (int rc = project_into(ctx, G_dev, dtype, n, ldg, ctx->d, 0, partial, P, false, ctx->stream)) return rc;
        CORE_CUDA(ctx, launch_aggregate(P, n, ctx->m, pbar_dev, ctx->stream));
    }
    if (int rc = apply_step_rule(ctx, rule, pbar_dev)) return rc;
    CORE_CUDA(ctx, launch_reconstruct(ctx->keys, ctx->t, pbar_dev, ctx->m, 0, ctx->d, out, ctx->sm_count, ctx->stream,
                                      epilogue));
    ctx->t += 1;
    return CORE_OK;
}

int core_round(core_ctx *ctx, const void *G_dev, int dtype, int32_t n, int64_t ldg, float *pbar_dev,
               float *gtilde_dev) {
    if (int rc = check_ctx(ctx)) return rc;
    if (!G_dev || !pbar_dev || !gtilde_dev || n < 1 || ldg < ctx->d || !valid_dtype(dtype)) return CORE_EINVAL;
    return round_with_epilogue(ctx, G_dev, dtype, n, ldg, pbar_dev, gtilde_dev, nullptr);
}

static int round_host_body(core_ctx *ctx, const void *G_host, int dtype, int32_t n, int64_t ldg, float *pbar_host,
                           float *gtilde_host);

int core_round_host(core_ctx *ctx, const void *G_host, int dtype, int32_t n, int64_t ldg, float *pbar_host,
                    float *gtilde_host) {
    if (int rc = check_ctx(ctx)) return rc;
    if (!G_host || !pbar_host || !gtilde_host || n < 1 || ldg < ctx->d || !valid_dtype(dtype)) return CORE_EINVAL;
    const int rc = round_host_body(ctx, G_host, dtype, n, ldg, pbar_host, gtilde_host);
    if (rc != CORE_OK && ctx->host_ready) {
        // copies enqueued before the failure may still be reading G_host or writing the outputs: the
        // caller gets its buffers back only once both streams have drained (a second error is ignored)
        const int first = ctx->last_cuda;
        cudaStreamSynchronize(ctx->work_stream);
        cudaStreamSynchronize(ctx->copy_stream);
        cudaGetLastError();
        ctx->last_cuda = first;
    }
    return rc;
}

static int round_host_body(core_ctx *ctx, const void *G_host, int dtype, int32_t n, int64_t ldg, float *pbar_host,
                           float *gtilde_host) {
    if (!ctx->host_ready) {
        // all or nothing: a half-made set of streams and events is torn down again
        cudaError_t e = cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        e = cudaStreamCreateWithFlags(&ctx->work_stream, cudaStreamNonBlocking);
        if (e != cudaSuccess) {
            cudaStreamDestroy(ctx->copy_stream);
            return cuda_fail(ctx, e);
        }
        cudaEvent_t *events[8] = {&ctx->in_ready[0], &ctx->in_ready[1], &ctx->in_free[0], &ctx->in_free[1],
                                  &ctx->out_ready[0], &ctx->out_ready[1], &ctx->out_free[0], &ctx->out_free[1]};
        int made = 0;
        for (; made < 8 && e == cudaSuccess; ++made) e = cudaEventCreateWithFlags(events[made], cudaEventDisableTiming);
        if (e != cudaSuccess) {
            for (int k = 0; k + 1 < made; ++k) cudaEventDestroy(*events[k]);
            cudaStreamDestroy(ctx->copy_stream);
            cudaStreamDestroy(ctx->work_stream);
            return cuda_fail(ctx, e);
        }
        ctx->host_ready = true;
    }
    const size_t es = elem_size(dtype);
    const int64_t d = ctx->d;
    // slab: a multiple of 4096 coordinates, about 64 MiB of input per slab over all machines
    int64_t slab = ((int64_t)64 << 20) / (int64_t)(es * (size_t)n);
    slab = slab / 4096 * 4096;
    if (slab < 4096) slab = 4096;
    if (slab > (d + 4095) / 4096 * 4096) slab = (d + 4095) / 4096 * 4096;
    const size_t in_bytes = round_up((size_t)n * (size_t)slab * es, 256);
    const size_t out_bytes = round_up((size_t)slab * sizeof(float), 256);
    const size_t need_slab = 2 * in_bytes + 2 * out_bytes;
    if (need_slab > ctx->slab_bytes) {
        if (ctx->slab) {
            cudaFree(ctx->slab);
            ctx->slab = nullptr;
            ctx->slab_bytes = 0;
        }
        cudaError_t e = core_malloc(&ctx->slab, need_slab);
        if (e != cudaSuccess) {
            cudaGetLastError();
            ctx->last_cuda = (int)e;
            return CORE_ENOMEM;
        }
        ctx->slab_bytes = need_slab;
    }
    const size_t pb = partial_bytes(ctx, n, slab, dtype);
    const size_t Pb = round_up((size_t)n * ctx->m * sizeof(float), 256);
    const size_t mb = round_up((size_t)ctx->m * sizeof(float), 256);
    if (int rc = ensure_workspace(ctx, pb + Pb + mb)) return rc;
    char *in_buf[2] = {static_cast<char *>(ctx->slab), static_cast<char *>(ctx->slab) + in_bytes};
    float *out_buf[2] = {reinterpret_cast<float *>(static_cast<char *>(ctx->slab) + 2 * in_bytes),
                         reinterpret_cast<float *>(static_cast<char *>(ctx->slab) + 2 * in_bytes + out_bytes)};
    float *partial = static_cast<float *>(ctx->ws);
    float *P = reinterpret_cast<float *>(static_cast<char *>(ctx->ws) + pb);
    float *pbar = reinterpret_cast<float *>(static_cast<char *>(ctx->ws) + pb + Pb);

    CORE_CUDA(ctx, cudaStreamSynchronize(ctx->stream));   // earlier work of the caller on this context

    // projection: slab s is copied while slab s-1 is projected
    const int64_t slabs = (d + slab - 1) / slab;
    for (int64_t s = 0; s < slabs; ++s) {
        const int b = (int)(s & 1);
        const int64_t k0 = s * slab;
        const int64_t len = d - k0 < slab ? d - k0 : slab;
        if (s >= 2) CORE_CUDA(ctx, cudaStreamWaitEvent(ctx->copy_stream, ctx->in_free[b], 0));
        for (int32_t i = 0; i < n; ++i)   // one copy per row: row strides may exceed the 2-D copy pitch limit
            CORE_CUDA(ctx, cudaMemcpyAsync(in_buf[b] + (size_t)i * (size_t)slab * es,
                                           static_cast<const char *>(G_host) + ((size_t)i * (size_t)ldg + (size_t)k0) * es,
                                           (size_t)len * es, cudaMemcpyHostToDevice, ctx->copy_stream));
        CORE_CUDA(ctx, cudaEventRecord(ctx->in_ready[b], ctx->copy_stream));
        CORE_CUDA(ctx, cudaStreamWaitEvent(ctx->work_stream, ctx->in_ready[b], 0));
        if (int rc = project_into(ctx, in_buf[b], dtype, n, slab, len, (uint64_t)k0 >> 2, partial, P, s > 0,
                                  ctx->work_stream))
            return rc;
        CORE_CUDA(ctx, cudaEventRecord(ctx->in_free[b], ctx->work_stream));
    }
    CORE_CUDA(ctx, launch_aggregate(P, n, ctx->m, pbar, ctx->work_stream));
    CORE_CUDA(ctx, cudaMemcpyAsync(pbar_host, pbar, (size_t)ctx->m * sizeof(float), cudaMemcpyDeviceToHost,
                                   ctx->work_stream));
    // reconstruction: slab s is copied back while slab s+1 is generated
    for (int64_t s = 0; s < slabs; ++s) {
        const int b = (int)(s & 1);
        const int64_t k0 = s * slab;
        const int64_t len = d - k0 < slab ? d - k0 : slab;
        if (s >= 2) CORE_CUDA(ctx, cudaStreamWaitEvent(ctx->work_stream, ctx->out_free[b], 0));
        CORE_CUDA(ctx, launch_reconstruct(ctx->keys, ctx->t, pbar, ctx->m, k0, k0 + len, out_buf[b], ctx->sm_count,
                                          ctx->work_stream));
        CORE_CUDA(ctx, cudaEventRecord(ctx->out_ready[b], ctx->work_stream));
        CORE_CUDA(ctx, cudaStreamWaitEvent(ctx->copy_stream, ctx->out_ready[b], 0));
        CORE_CUDA(ctx, cudaMemcpyAsync(gtilde_host + k0, out_buf[b], (size_t)len * sizeof(float),
                                       cudaMemcpyDeviceToHost, ctx->copy_stream));
        CORE_CUDA(ctx, cudaEventRecord(ctx->out_free[b], ctx->copy_stream));
    }
    CORE_CUDA(ctx, cudaStreamSynchronize(ctx->work_stream));
    CORE_CUDA(ctx, cudaStreamSynchronize(ctx->copy_stream));
    ctx->t += 1;
    return CORE_OK;
}

/* ---- least squares ---------------------------------------------------------- */

int core_ls_create(core_ls **out, const float *A_dev, const float *b_dev, int32_t n, int32_t rows, int64_t d) {
    if (!out) return CORE_EINVAL;
    *out = nullptr;
    if (!A_dev || !b_dev || n < 1 || rows < 1 || d < 1) return CORE_EINVAL;
    core_ls *ls = new (std::nothrow) core_ls();
    if (!ls) return CORE_ENOMEM;
    ls->A = A_dev;
    ls->b = b_dev;
    ls->n = n;
    ls->rows = rows;
    ls->d = d;
    int sm = 0;
    cudaError_t e = cudaGetDevice(&ls->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, ls->device);
    if (e != cudaSuccess) {
        delete ls;
        return CORE_ECUDA;
    }
    ls->plan = make_ls_plan(n, rows, d, sm);
    ls->fused_plan = make_ls_fused_plan(n, rows, d, sm);
    const int max_splits = ls->plan.splits > ls->fused_plan.splits ? ls->plan.splits : ls->fused_plan.splits;
    const size_t res_b = round_up((size_t)n * rows * sizeof(float), 256);
    const size_t part_b = round_up((size_t)n * max_splits * (size_t)d * sizeof(float), 256);
    const size_t G_b = round_up((size_t)n * (size_t)d * sizeof(float), 256);
    const size_t gt_b = round_up((size_t)d * sizeof(float), 256);
    const size_t scalars_b = 256;                          // trial loss (double) and acceptance flag
    char *base = nullptr;
    e = core_malloc(reinterpret_cast<void **>(&base), res_b + part_b + G_b + gt_b + scalars_b);
    if (e != cudaSuccess) {
        cudaGetLastError();
        delete ls;
        return CORE_ENOMEM;
    }
    ls->res = reinterpret_cast<float *>(base);
    ls->part = reinterpret_cast<float *>(base + res_b);
    ls->G = reinterpret_cast<float *>(base + res_b + part_b);
    ls->y = reinterpret_cast<float *>(base + res_b + part_b + G_b);
    ls->f_trial = reinterpret_cast<double *>(base + res_b + part_b + G_b + gt_b);
    ls->accepted = reinterpret_cast<int *>(base + res_b + part_b + G_b + gt_b + 16);
    ls->step = reinterpret_cast<float *>(base + res_b + part_b + G_b + gt_b + 32);
    *out = ls;
    return CORE_OK;
}

int core_ls_destroy(core_ls *ls) {
    if (!ls) return CORE_EINVAL;
    const int rc = cudaFree(ls->res) == cudaSuccess ? CORE_OK : CORE_ECUDA;   // res is the base of the block
    delete ls;
    return rc;
}

static int ls_gradients_into(core_ctx *ctx, core_ls *ls, const float *x_dev, float *G) {
    if (ls_fused_usable(ls->fused_plan, ls->A, x_dev, ls->part)) {
        // single pass over A: residual and A^T r per row range, then the fixed-order reduce
        CORE_CUDA(ctx, launch_ls_fused(ls->fused_plan, ls->A, ls->b, x_dev, ls->n, ls->rows, ls->d, ls->part,
                                       ctx->stream));
        CORE_CUDA(ctx, launch_ls_reduce(ls->fused_plan, ls->part, ls->n, ls->rows, ls->d, G, ctx->stream));
        return CORE_OK;
    }
    CORE_CUDA(ctx, launch_ls_residual(ls->A, ls->b, x_dev, ls->n, ls->rows, ls->d, ls->res, ctx->stream));
    CORE_CUDA(ctx, launch_ls_at_r(ls->plan, ls->A, ls->res, ls->n, ls->rows, ls->d, ls->part, ctx->stream));
    CORE_CUDA(ctx, launch_ls_reduce(ls->plan, ls->part, ls->n, ls->rows, ls->d, G, ctx->stream));
    return CORE_OK;
}

// Gradients at x_eval, then the round with the given epilogue.  Where the single-pass gradient kernel
// and the scalar projection both apply, the projection sums the per-row-range partial gradients while
// it stages its tiles, so the machine gradients G are never written or read back.
static int ls_round(core_ctx *ctx, core_ls *ls, const float *x_eval, float *out, const ReconstructEpilogue *epilogue,
                    const StepRule *rule = nullptr) {
    if (ls->n <= kMaxGroup && ls_fused_usable(ls->fused_plan, ls->A, x_eval, ls->part)) {
        const ProjectPlan plan = make_project_plan(ls->n, ctx->m, ctx->d, CORE_F32, ctx->sm_count);
        if (plan.mma == 0) {
            if (int rc = ensure_workspace(ctx, partial_bytes(ctx, ls->n, ctx->d, CORE_F32))) return rc;
            float *partial = static_cast<float *>(ctx->ws);
            CORE_CUDA(ctx, launch_ls_fused(ls->fused_plan, ls->A, ls->b, x_eval, ls->n, ls->rows, ls->d, ls->part,
                                           ctx->stream));
            CORE_CUDA(ctx, launch_project(plan, ctx->keys, ctx->t, ls->part, CORE_F32, ls->n, ls->d, ctx->d, ctx->m, 0,
                                          partial, ctx->stream, ls->fused_plan.splits, 1.0f / (float)ls->rows));
            CORE_CUDA(ctx, launch_finish_aggregate(partial, plan.grid_x, ls->n, ctx->m, ctx->pbar, ctx->stream));
            if (int rc = apply_step_rule(ctx, rule, ctx->pbar)) return rc;
            CORE_CUDA(ctx, launch_reconstruct(ctx->keys, ctx->t, ctx->pbar, ctx->m, 0, ctx->d, out, ctx->sm_count,
                                              ctx->stream, epilogue));
            ctx->t += 1;
            return CORE_OK;
        }
    }
    if (int rc = ls_gradients_into(ctx, ls, x_eval, ls->G)) return rc;
    return round_with_epilogue(ctx, ls->G, CORE_F32, ls->n, ls->d, ctx->pbar, out, epilogue, rule);
}

int core_ls_gradients(core_ctx *ctx, core_ls *ls, const float *x_dev, float *G_out_dev) {
    if (int rc = check_ctx(ctx)) return rc;
    if (!ls || !x_dev || !G_out_dev || ls->d != ctx->d || ls->device != ctx->device) return CORE_EINVAL;
    return ls_gradients_into(ctx, ls, x_dev, G_out_dev);
}

int core_gd_step(core_ctx *ctx, core_ls *ls, float h, float *x_dev) {
    if (int rc = check_ctx(ctx)) return rc;
    if (!ls || !x_dev || ls->d != ctx->d || ls->device != ctx->device) return CORE_EINVAL;
    // x <- x - h * gtilde inside the reconstruction: the estimate is never stored
    const ReconstructEpilogue update{x_dev, h, nullptr, nullptr};
    return ls_round(ctx, ls, x_dev, x_dev, &update);
}

int core_agd_step(core_ctx *ctx, core_ls *ls, float h, float beta, float *x_dev, float *x_prev_dev) {
    if (int rc = check_ctx(ctx)) return rc;
    if (!ls || !x_dev || !x_prev_dev || x_dev == x_prev_dev || ls->d != ctx->d || ls->device != ctx->device)
        return CORE_EINVAL;
    CORE_CUDA(ctx, launch_lookahead(x_dev, x_prev_dev, 1.0f - beta, ls->d, ls->y, ctx->stream));
    // x_prev <- x and x <- y - h * gtilde(y), both inside the reconstruction
    const ReconstructEpilogue update{ls->y, h, x_dev, x_prev_dev};
    return ls_round(ctx, ls, ls->y, x_dev, &update);
}

int core_gd_step_guarded(core_ctx *ctx, core_ls *ls, float h, float *x_dev, double *f_dev, int32_t *accepted_dev) {
    if (int rc = check_ctx(ctx)) return rc;
    if (!ls || !x_dev || !f_dev || ls->d != ctx->d || ls->device != ctx->device) return CORE_EINVAL;
    // trial point y = x - h * gtilde, written by the reconstruction; x is left untouched
    const ReconstructEpilogue trial{x_dev, h, nullptr, nullptr};
    if (int rc = ls_round(ctx, ls, x_dev, ls->y, &trial)) return rc;
    CORE_CUDA(ctx, launch_ls_residual(ls->A, ls->b, ls->y, ls->n, ls->rows, ls->d, ls->res, ctx->stream));
    CORE_CUDA(ctx, launch_ls_loss(ls->res, ls->n, ls->rows, ls->f_trial, ctx->stream));
    // decided on the device: no host synchronisation inside the step
    CORE_CUDA(ctx, launch_keep_better(ls->f_trial, ls->y, ls->d, f_dev, x_dev, ls->accepted, accepted_dev,
                                      ctx->stream));
    return CORE_OK;
}

int core_gd_step_option1(core_ctx *ctx, core_ls *ls, double r1, double H, double c, float *x_dev, double *f_dev,
                         int32_t *accepted_dev, float *p_dev, float *h_dev) {
    if (int rc = check_ctx(ctx)) return rc;
    if (!ls || !x_dev || !f_dev || ls->d != ctx->d || ls->device != ctx->device || !(r1 > 0.0) || !(H > 0.0) ||
        !(c > 0.0))
        return CORE_EINVAL;
    // the step is formed on the device between aggregation and reconstruction; the reconstruction reads it
    // there and writes the trial point y = x - h * gtilde; x is left untouched until the comparison
    const StepRule rule{r1, H, c, ls->step + 1, ls->step};
    ReconstructEpilogue trial{x_dev, 0.f, nullptr, nullptr};
    trial.step_dev = ls->step;
    if (int rc = ls_round(ctx, ls, x_dev, ls->y, &trial, &rule)) return rc;
    CORE_CUDA(ctx, launch_ls_residual(ls->A, ls->b, ls->y, ls->n, ls->rows, ls->d, ls->res, ctx->stream));
    CORE_CUDA(ctx, launch_ls_loss(ls->res, ls->n, ls->rows, ls->f_trial, ctx->stream));
    CORE_CUDA(ctx, launch_keep_better(ls->f_trial, ls->y, ls->d, f_dev, x_dev, ls->accepted, accepted_dev,
                                      ctx->stream));
    if (h_dev)
        CORE_CUDA(ctx, cudaMemcpyAsync(h_dev, ls->step, sizeof(float), cudaMemcpyDeviceToDevice, ctx->stream));
    if (p_dev)
        CORE_CUDA(ctx, cudaMemcpyAsync(p_dev, ls->step + 1, sizeof(float), cudaMemcpyDeviceToDevice, ctx->stream));
    return CORE_OK;
}

int core_gossip_round(core_ctx *ctx, const float *W_dev, const float *P_in_dev, int32_t n, float *P_out_dev) {
    if (int rc = check_ctx(ctx)) return rc;
    if (!W_dev || !P_in_dev || !P_out_dev || P_in_dev == P_out_dev || n < 1) return CORE_EINVAL;
    CORE_CUDA(ctx, launch_gossip_round(W_dev, P_in_dev, n, ctx->m, P_out_dev, ctx->stream));
    return CORE_OK;
}

int core_decentralized_step(core_ctx *ctx, core_ls *ls, const float *W_dev, int32_t rounds, int32_t reader,
                            int as_printed, float h, float *x_dev, float *spread_dev) {
    if (int rc = check_ctx(ctx)) return rc;
    if (!ls || !W_dev || !x_dev || ls->d != ctx->d || ls->device != ctx->device || rounds < 0 || reader < 0 ||
        reader >= ls->n)
        return CORE_EINVAL;
    const int32_t n = ls->n;
    const size_t pb = partial_bytes(ctx, n, ctx->d, CORE_F32);
    const size_t Pb = round_up((size_t)n * ctx->m * sizeof(float), 256);
    if (int rc = ensure_workspace(ctx, pb + 2 * Pb)) return rc;
    float *partial = static_cast<float *>(ctx->ws);
    float *P = reinterpret_cast<float *>(static_cast<char *>(ctx->ws) + pb);
    float *P_next = reinterpret_cast<float *>(static_cast<char *>(ctx->ws) + pb + Pb);
    // every machine projects its own gradient; nothing is combined centrally
    if (int rc = ls_gradients_into(ctx, ls, x_dev, ls->G)) return rc;
    if (int rc = project_into(ctx, ls->G, CORE_F32, n, ls->d, ctx->d, 0, partial, P, false, ctx->stream)) return rc;
    // the m-dimensional averaging problem, by gossip with the neighbours: row i is machine i's estimate
    for (int32_t r = 0; r < rounds; ++r) {
        CORE_CUDA(ctx, launch_gossip_round(W_dev, P, n, ctx->m, P_next, ctx->stream));
        float *swap = P;
        P = P_next;
        P_next = swap;
    }
    if (spread_dev) CORE_CUDA(ctx, launch_consensus_spread(P, n, ctx->m, reader, spread_dev, ctx->stream));
    // reconstruction from the reader's estimate, update inside the kernel; the printed prefactor n/m is
    // the mean convention's 1/m with an n times longer step
    const ReconstructEpilogue update{x_dev, as_printed ? h * (float)n : h, nullptr, nullptr};
    CORE_CUDA(ctx, launch_reconstruct(ctx->keys, ctx->t, P + (size_t)reader * ctx->m, ctx->m, 0, ctx->d, x_dev,
                                      ctx->sm_count, ctx->stream, &update));
    ctx->t += 1;
    return CORE_OK;
}

int core_ls_loss(core_ctx *ctx, core_ls *ls, const float *x_dev, double *loss_dev) {
    if (int rc = check_ctx(ctx)) return rc;
    if (!ls || !x_dev || !loss_dev || ls->d != ctx->d || ls->device != ctx->device) return CORE_EINVAL;
    CORE_CUDA(ctx, launch_ls_residual(ls->A, ls->b, x_dev, ls->n, ls->rows, ls->d, ls->res, ctx->stream));
    CORE_CUDA(ctx, launch_ls_loss(ls->res, ls->n, ls->rows, loss_dev, ctx->stream));
    return CORE_OK;
}

int core_ls_loss_host(core_ctx *ctx, core_ls *ls, const float *x_dev, double *loss_host) {
    if (int rc = check_ctx(ctx)) return rc;
    if (!ls || !x_dev || !loss_host || ls->d != ctx->d || ls->device != ctx->device) return CORE_EINVAL;
    CORE_CUDA(ctx, launch_ls_residual(ls->A, ls->b, x_dev, ls->n, ls->rows, ls->d, ls->res, ctx->stream));
    CORE_CUDA(ctx, launch_ls_loss(ls->res, ls->n, ls->rows, ls->f_trial, ctx->stream));
    CORE_CUDA(ctx, cudaMemcpyAsync(loss_host, ls->f_trial, sizeof(double), cudaMemcpyDeviceToHost, ctx->stream));
    return CORE_OK;
}

/* ---- run-time diagnostics ------------------------------------------------------ */

int core_debug_force_project_kernel(int kind) {
    if (kind < -1 || kind > 2) return CORE_EINVAL;
    project_force_kernel(kind);
    return CORE_OK;
}

int core_debug_fail_allocations(int count) {
    if (count < 0) return CORE_EINVAL;
    g_fail_allocations.store(count);
    return CORE_OK;
}

int core_debug_wait_timeout(uint32_t limit_us, int32_t code, uint32_t observed_host[2]) {
    if (!observed_host || limit_us < 1 || limit_us > 100000 || code < 1) return CORE_EINVAL;
    uint32_t *observed = nullptr;
    if (core_malloc(reinterpret_cast<void **>(&observed), 2 * sizeof(uint32_t)) != cudaSuccess) {
        cudaGetLastError();
        return CORE_ENOMEM;
    }
    cudaError_t e = cudaMemset(observed, 0xFF, 2 * sizeof(uint32_t));
    if (e == cudaSuccess) e = launch_wait_timeout_probe((uint64_t)limit_us * 1000ull, code, observed, nullptr);
    if (e == cudaSuccess) e = cudaMemcpy(observed_host, observed, 2 * sizeof(uint32_t), cudaMemcpyDeviceToHost);
    cudaFree(observed);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return CORE_ECUDA;
    }
    return CORE_OK;
}

/* ---- generator windows -------------------------------------------------------- */

int core_debug_philox(core_ctx *ctx, uint32_t j, uint64_t q0, int64_t nq, uint32_t *words_dev) {
    if (int rc = check_ctx(ctx)) return rc;
    if (!words_dev || nq < 0 || (reinterpret_cast<uintptr_t>(words_dev) % 16) != 0) return CORE_EINVAL;
    CORE_CUDA(ctx, launch_debug_philox(ctx->keys, ctx->t, j, q0, nq, words_dev, ctx->stream));
    return CORE_OK;
}

int core_debug_gaussians(core_ctx *ctx, uint32_t j, uint64_t q0, int64_t nq, float *z_dev) {
    if (int rc = check_ctx(ctx)) return rc;
    if (!z_dev || nq < 0 || (reinterpret_cast<uintptr_t>(z_dev) % 16) != 0) return CORE_EINVAL;
    CORE_CUDA(ctx, launch_debug_gaussians(ctx->keys, ctx->t, j, q0, nq, z_dev, ctx->stream));
    return CORE_OK;
}

int core_debug_box_muller(core_ctx *ctx, const uint32_t *words_dev, int64_t nb, float *z_dev) {
    if (int rc = check_ctx(ctx)) return rc;
    if (!words_dev || !z_dev || nb < 0 || (reinterpret_cast<uintptr_t>(words_dev) % 16) != 0 ||
        (reinterpret_cast<uintptr_t>(z_dev) % 16) != 0)
        return CORE_EINVAL;
    CORE_CUDA(ctx, launch_debug_box_muller(words_dev, nb, z_dev, ctx->stream));
    return CORE_OK;
}

int core_debug_project_plan(int32_t n, int32_t m, int64_t d, int dtype, int32_t sm_count, int64_t out[10]) {
    if (!out || n < 1 || m < 1 || d < 1 || sm_count < 1 || !valid_dtype(dtype)) return CORE_EINVAL;
    const ProjectPlan p = make_project_plan(project_group(n, m), m, d, dtype, sm_count);
    const int64_t v[10] = {p.nb, p.jt, p.uq, p.tile_q, p.tj, p.tq, p.grid_x, p.grid_y, p.tiles, (int64_t)p.smem};
    for (int i = 0; i < 10; ++i) out[i] = v[i];
    return CORE_OK;
}

}  // extern "C"
