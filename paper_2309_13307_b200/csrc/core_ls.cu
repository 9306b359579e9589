// Machine gradients of the least-squares objective that drives Algorithm 2:
// f_i(x) = 1/(2 rows) ||A_i x - b_i||^2, g_i = A_i^T (A_i x - b_i) / rows.
// Two streaming passes over A (both HBM-bound), every sum in a fixed order.
#include "core_internal.h"

namespace core {

namespace {

constexpr int kLsThreads = 256;
constexpr int kStrip = kLsThreads * 4;   // columns per CTA in the A^T r pass

// One warp per row: res = A[row] . x - b[row].
__global__ void __launch_bounds__(kLsThreads)
ls_residual_kernel(const float *__restrict__ A, const float *__restrict__ b, const float *__restrict__ x,
                   int64_t total_rows, int64_t d, int vec_ok, float *__restrict__ res) {
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (kLsThreads / 32) + (threadIdx.x >> 5);
    if (row >= total_rows) return;
    const float *a = A + row * d;
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
    if (vec_ok) {
        const float4 *a4 = reinterpret_cast<const float4 *>(a);
        const float4 *x4 = reinterpret_cast<const float4 *>(x);
        const int64_t n4 = d >> 2;
        for (int64_t c = lane; c < n4; c += 32) {
            const float4 av = __ldcs(a4 + c);     // A is streamed: read once per pass
            const float4 xv = __ldg(x4 + c);
            s0 = fmaf(av.x, xv.x, s0);
            s1 = fmaf(av.y, xv.y, s1);
            s2 = fmaf(av.z, xv.z, s2);
            s3 = fmaf(av.w, xv.w, s3);
        }
    } else {
        for (int64_t k = lane; k < d; k += 32) s0 = fmaf(a[k], __ldg(x + k), s0);
    }
    float s = (s0 + s1) + (s2 + s3);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
    if (lane == 0) res[row] = s - b[row];
}

// CTA (strip, split, machine): columns [strip*kStrip, +kStrip), rows of range `split`.
__global__ void __launch_bounds__(kLsThreads)
ls_at_r_kernel(const float *__restrict__ A, const float *__restrict__ res, int rows, int64_t d, int splits,
               int rows_per_split, int vec_ok, float *__restrict__ part) {
    const int i = blockIdx.z, s = blockIdx.y;
    const int64_t k0 = (int64_t)blockIdx.x * kStrip + threadIdx.x * 4;
    const int r_begin = s * rows_per_split;
    const int r_end = min(r_begin + rows_per_split, rows);
    const float *Ai = A + (int64_t)i * rows * d;
    const float *ri = res + (int64_t)i * rows;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (vec_ok && k0 + 4 <= d) {
        int r = r_begin;
        for (; r + 4 <= r_end; r += 4) {          // four rows in flight
            float4 av[4];
            float rv[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                av[u] = __ldcs(reinterpret_cast<const float4 *>(Ai + (int64_t)(r + u) * d + k0));
                rv[u] = __ldg(ri + r + u);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                acc.x = fmaf(av[u].x, rv[u], acc.x);
                acc.y = fmaf(av[u].y, rv[u], acc.y);
                acc.z = fmaf(av[u].z, rv[u], acc.z);
                acc.w = fmaf(av[u].w, rv[u], acc.w);
            }
        }
        for (; r < r_end; ++r) {
            const float4 av = __ldcs(reinterpret_cast<const float4 *>(Ai + (int64_t)r * d + k0));
            const float rv = __ldg(ri + r);
            acc.x = fmaf(av.x, rv, acc.x);
            acc.y = fmaf(av.y, rv, acc.y);
            acc.z = fmaf(av.z, rv, acc.z);
            acc.w = fmaf(av.w, rv, acc.w);
        }
        *reinterpret_cast<float4 *>(part + ((int64_t)i * splits + s) * d + k0) = acc;
    } else {
        float v[4] = {0.f, 0.f, 0.f, 0.f};
        for (int r = r_begin; r < r_end; ++r) {
            const float rv = __ldg(ri + r);
#pragma unroll
            for (int l = 0; l < 4; ++l)
                if (k0 + l < d) v[l] = fmaf(Ai[(int64_t)r * d + k0 + l], rv, v[l]);
        }
#pragma unroll
        for (int l = 0; l < 4; ++l)
            if (k0 + l < d) part[((int64_t)i * splits + s) * d + k0 + l] = v[l];
    }
}

__global__ void ls_reduce_kernel(const float *__restrict__ part, int n, int splits, int64_t d, float inv_rows,
                                 float *__restrict__ G) {
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (int64_t)n * d) return;
    const int i = (int)(idx / d);
    const int64_t k = idx % d;
    float s = 0.f;
    for (int c = 0; c < splits; ++c) s += part[((int64_t)i * splits + c) * d + k];
    G[idx] = s * inv_rows;
}

// One CTA; thread t sums residual squares t, t+256, ... in double, then a fixed tree.
__global__ void __launch_bounds__(kLsThreads)
ls_loss_kernel(const float *__restrict__ res, int64_t total, double scale, double *loss) {
    __shared__ double sh[kLsThreads];
    double s = 0.0;
    for (int64_t r = threadIdx.x; r < total; r += kLsThreads) {
        const double v = (double)res[r];
        s += v * v;
    }
    sh[threadIdx.x] = s;
    __syncthreads();
    for (int off = kLsThreads / 2; off > 0; off >>= 1) {
        if ((int)threadIdx.x < off) sh[threadIdx.x] += sh[threadIdx.x + off];
        __syncthreads();
    }
    if (threadIdx.x == 0) loss[0] = sh[0] * scale;
}

// ---- single pass over A (rows of up to 8192 columns) -------------------------------------
// A CTA owns a range of rows of one machine.  Thread t keeps x and its partial gradient for the
// columns {4(t + 256c) .. +3, c < C4} in registers.  Rows are prefetched with cp.async into a ring in
// shared memory, every thread copying exactly the 16-byte pieces it will read back itself, so the
// ring needs no barrier; the only barrier per row is the one of the dot-product reduction.
// For row r: res = A[r].x - b[r] (fixed-order reduction), then acc += res * A[r] from the same
// registers.  A is read from HBM once; the partial gradients of the CTAs of a machine are added by
// ls_reduce_kernel in ascending order.
constexpr int kRing = 4;   // rows in flight per CTA

__device__ __forceinline__ void ls_cp_async16(void *smem_dst, const void *gmem_src) {
    const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gmem_src) : "memory");
}

template <int C4>
__global__ void __launch_bounds__(kLsThreads, 1)
ls_fused_kernel(const float *__restrict__ A, const float *__restrict__ b, const float *__restrict__ x, int rows,
                int d4, int splits, int rows_per_split, float *__restrict__ part) {
    extern __shared__ __align__(16) unsigned char ls_smem[];
    float4 *ring = reinterpret_cast<float4 *>(ls_smem);                       // kRing x (C4 * 256) float4
    float *warp_sums = reinterpret_cast<float *>(ring + kRing * C4 * kLsThreads);   // 2 x 8
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int i = blockIdx.y, s = blockIdx.x;
    const int r_begin = s * rows_per_split;
    const int r_end = min(r_begin + rows_per_split, rows);
    const float4 *Ai = reinterpret_cast<const float4 *>(A) + (int64_t)i * rows * d4;
    const float *bi = b + (int64_t)i * rows;

    float4 xv[C4], acc[C4];
#pragma unroll
    for (int c = 0; c < C4; ++c) {
        const int col = tid + c * kLsThreads;
        xv[c] = col < d4 ? __ldg(reinterpret_cast<const float4 *>(x) + col) : make_float4(0.f, 0.f, 0.f, 0.f);
        acc[c] = make_float4(0.f, 0.f, 0.f, 0.f);
    }

    auto prefetch = [&](int r) {
        if (r < r_end) {
            float4 *slot = ring + (size_t)((r - r_begin) % kRing) * C4 * kLsThreads;
            const float4 *row = Ai + (int64_t)r * d4;
#pragma unroll
            for (int c = 0; c < C4; ++c) {
                const int col = tid + c * kLsThreads;
                if (col < d4) ls_cp_async16(slot + col, row + col);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");      // one group per row, empty past the end
    };

#pragma unroll
    for (int p = 0; p < kRing - 1; ++p) prefetch(r_begin + p);

    for (int r = r_begin; r < r_end; ++r) {
        prefetch(r + kRing - 1);
        asm volatile("cp.async.wait_group %0;" ::"n"(kRing - 1) : "memory");   // row r has landed (own pieces)
        const float4 *slot = ring + (size_t)((r - r_begin) % kRing) * C4 * kLsThreads;
        float4 av[C4];
        float p0 = 0.f, p1 = 0.f, p2 = 0.f, p3 = 0.f;
#pragma unroll
        for (int c = 0; c < C4; ++c) {
            const int col = tid + c * kLsThreads;
            av[c] = col < d4 ? slot[col] : make_float4(0.f, 0.f, 0.f, 0.f);
            p0 = fmaf(av[c].x, xv[c].x, p0);
            p1 = fmaf(av[c].y, xv[c].y, p1);
            p2 = fmaf(av[c].z, xv[c].z, p2);
            p3 = fmaf(av[c].w, xv[c].w, p3);
        }
        float p = (p0 + p1) + (p2 + p3);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) p += __shfl_xor_sync(0xFFFFFFFFu, p, off);
        float *sums = warp_sums + ((r - r_begin) & 1) * (kLsThreads / 32);
        if (lane == 0) sums[warp] = p;
        __syncthreads();
        float dot = 0.f;
#pragma unroll
        for (int w = 0; w < kLsThreads / 32; ++w) dot += sums[w];
        const float res = dot - __ldg(bi + r);
#pragma unroll
        for (int c = 0; c < C4; ++c) {
            acc[c].x = fmaf(av[c].x, res, acc[c].x);
            acc[c].y = fmaf(av[c].y, res, acc[c].y);
            acc[c].z = fmaf(av[c].z, res, acc[c].z);
            acc[c].w = fmaf(av[c].w, res, acc[c].w);
        }
    }
    float4 *out = reinterpret_cast<float4 *>(part) + ((int64_t)i * splits + s) * d4;
#pragma unroll
    for (int c = 0; c < C4; ++c) {
        const int col = tid + c * kLsThreads;
        if (col < d4) out[col] = acc[c];
    }
}

// Comparison step of Algorithm 3: one thread decides, then every thread copies if told to.
__global__ void keep_better_decide_kernel(const double *__restrict__ f_trial, double *__restrict__ f,
                                          int *__restrict__ flag, int32_t *__restrict__ flag_out) {
    const int take = *f_trial < *f ? 1 : 0;     // a tie keeps the current point
    if (take) *f = *f_trial;
    *flag = take;
    if (flag_out) *flag_out = take;
}

__global__ void keep_better_copy_kernel(const int *__restrict__ flag, const float *__restrict__ trial, int64_t d,
                                        float *__restrict__ x) {
    if (*flag == 0) return;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; k < d; k += stride) x[k] = trial[k];
}

bool vec_ok_for(const float *A, int64_t d) {
    return (reinterpret_cast<uintptr_t>(A) % 16) == 0 && d % 4 == 0;
}

}  // namespace

cudaError_t launch_keep_better(const double *f_trial, const float *trial, int64_t d, double *f, float *x,
                               int *flag_scratch, int32_t *flag_out, cudaStream_t stream) {
    keep_better_decide_kernel<<<1, 1, 0, stream>>>(f_trial, f, flag_scratch, flag_out);
    int64_t blocks = (d + 255) / 256;
    if (blocks > 148 * 8) blocks = 148 * 8;
    keep_better_copy_kernel<<<(unsigned)blocks, 256, 0, stream>>>(flag_scratch, trial, d, x);
    return cudaGetLastError();
}

LsPlan make_ls_fused_plan(int32_t n, int32_t rows, int64_t d, int sm_count) {
    LsPlan p{};
    if (d % 4 != 0 || d > 4 * 8 * kLsThreads) return p;     // splits == 0: not available
    int per_machine = sm_count / n;                          // one CTA per SM, machines side by side
    if (per_machine < 1) per_machine = 1;
    if (per_machine > rows) per_machine = rows;
    p.rows_per_split = (rows + per_machine - 1) / per_machine;
    p.splits = (rows + p.rows_per_split - 1) / p.rows_per_split;
    return p;
}

cudaError_t launch_ls_fused(const LsPlan &plan, const float *A, const float *b, const float *x, int32_t n,
                            int32_t rows, int64_t d, float *part, cudaStream_t stream) {
    const int d4 = (int)(d / 4);
    int c4 = 1;
    while (c4 * kLsThreads < d4) c4 *= 2;
    const size_t smem = (size_t)kRing * c4 * kLsThreads * 16 + 2 * (kLsThreads / 32) * sizeof(float);
    dim3 grid(plan.splits, n);
    auto go = [&](auto kernel) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kernel<<<grid, kLsThreads, smem, stream>>>(A, b, x, rows, d4, plan.splits, plan.rows_per_split, part);
        return cudaGetLastError();
    };
    switch (c4) {
        case 1: return go(ls_fused_kernel<1>);
        case 2: return go(ls_fused_kernel<2>);
        case 4: return go(ls_fused_kernel<4>);
        default: return go(ls_fused_kernel<8>);
    }
}

bool ls_fused_usable(const LsPlan &fused_plan, const float *A, const float *x, const float *part) {
    return fused_plan.splits > 0 && ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(x) |
                                      reinterpret_cast<uintptr_t>(part)) % 16) == 0;
}

LsPlan make_ls_plan(int32_t n, int32_t rows, int64_t d, int sm_count) {
    LsPlan p{};
    const int64_t strips = (d + kStrip - 1) / kStrip;
    // aim at about eight CTAs per SM so that enough loads are in flight
    int64_t want = ((int64_t)sm_count * 8 + n * strips - 1) / (n * strips);
    if (want < 1) want = 1;
    if (want > rows) want = rows;
    if (want > 64) want = 64;
    p.rows_per_split = (int)((rows + want - 1) / want);
    p.splits = (rows + p.rows_per_split - 1) / p.rows_per_split;
    return p;
}

cudaError_t launch_ls_residual(const float *A, const float *b, const float *x, int32_t n, int32_t rows,
                               int64_t d, float *res, cudaStream_t stream) {
    const int64_t total = (int64_t)n * rows;
    const int warps = kLsThreads / 32;
    const int vec = vec_ok_for(A, d) && (reinterpret_cast<uintptr_t>(x) % 16) == 0;
    ls_residual_kernel<<<(unsigned)((total + warps - 1) / warps), kLsThreads, 0, stream>>>(A, b, x, total, d,
                                                                                         vec, res);
    return cudaGetLastError();
}

cudaError_t launch_ls_at_r(const LsPlan &plan, const float *A, const float *res, int32_t n, int32_t rows,
                           int64_t d, float *part, cudaStream_t stream) {
    dim3 grid((unsigned)((d + kStrip - 1) / kStrip), plan.splits, n);
    const int vec = vec_ok_for(A, d) && (reinterpret_cast<uintptr_t>(part) % 16) == 0;
    ls_at_r_kernel<<<grid, kLsThreads, 0, stream>>>(A, res, rows, d, plan.splits, plan.rows_per_split, vec, part);
    return cudaGetLastError();
}

cudaError_t launch_ls_reduce(const LsPlan &plan, const float *part, int32_t n, int32_t rows, int64_t d,
                             float *G, cudaStream_t stream) {
    const int64_t total = (int64_t)n * d;
    ls_reduce_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(part, n, plan.splits, d,
                                                                         1.0f / (float)rows, G);
    return cudaGetLastError();
}

cudaError_t launch_ls_loss(const float *res, int32_t n, int32_t rows, double *loss, cudaStream_t stream) {
    ls_loss_kernel<<<1, kLsThreads, 0, stream>>>(res, (int64_t)n * rows, 1.0 / (2.0 * (double)rows * (double)n),
                                                 loss);
    return cudaGetLastError();
}

}  // namespace core
