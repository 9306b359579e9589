// Fused regenerate-and-reconstruct kernel: gtilde[k] = (1/m) sum_j pbar[j] xi_j[k]
// (Algorithm 1, receiver's step; the equation that follows Algorithm 1).
//
// A thread owns UQ coordinate blocks of four coordinates and runs over all vectors j,
// regenerating xi_j for its blocks from the same counters the projection used.  The
// part of the Philox evaluation that depends only on the block is computed once per
// thread; the part that depends only on j is tabulated per CTA in shared memory next
// to pbar[j], so the loop reads one 16-byte broadcast per j.  Every output coordinate
// is written exactly once, as a 16-byte store where alignment allows.
#include "core_internal.h"

namespace core {

namespace {

constexpr int kRecUQ = 2;                         // coordinate blocks per thread per group
constexpr int kGroupQ = kThreads * kRecUQ;        // blocks per CTA step
constexpr int kJChunk = 2048;                     // vectors tabulated at a time (32 KB)

struct ReconstructArgs {
    const float *pbar;
    float *out;
    int64_t k_begin;
    int64_t k_end;
    int m;
    int vec_ok;       // out (and the epilogue arrays) + 4*(q - q_begin) are 16-byte aligned
    uint32_t t;
    RoundKeys keys;
    ReconstructEpilogue epi;   // base == nullptr: store the estimate itself
};

constexpr int kRecJStep = 2;                      // vectors generated together per loop step

// acc[u] += sum over JS consecutive table entries of pbar[j] * xi_j[block u], j ascending.
template <int JS, int UQ>
__device__ __forceinline__ void rec_step(const uint4 *entries, const QPart (&qp)[UQ], const RoundKeys &keys,
                                         float4 (&acc)[UQ]) {
    constexpr int kRecUQ = UQ;
    uint4 w[JS * kRecUQ];
    float p[JS];
#pragma unroll
    for (int s = 0; s < JS; ++s) {
        const uint4 e = entries[s];
        p[s] = __uint_as_float(e.w);
        JPart jp;
        jp.x0 = e.x;
        jp.x2 = e.y;
        jp.w3 = e.z;
#pragma unroll
        for (int u = 0; u < kRecUQ; ++u) w[s * kRecUQ + u] = philox_combine(jp, qp[u], keys);
    }
    BmParts r[JS * kRecUQ];
    box_muller_parts<JS * kRecUQ>(w, r);
    // pbar_j xi_j with the message meeting the radius first: ((pbar S) y) sp and (pbar S) cs, four packed
    // instructions per call instead of five, and xi_j itself (pbar = 1) bit for bit what the projection
    // multiplies with.  Accumulator lanes: (x, z) = cosine lanes of pair a, b; (y, w) = sine lanes.
#pragma unroll
    for (int s = 0; s < JS; ++s) {
#pragma unroll
        for (int u = 0; u < kRecUQ; ++u) {
            const BmParts rr = r[s * kRecUQ + u];
            const float2 ps = __fmul2_rn(make_float2(p[s], p[s]), rr.s);
            const float2 psy = __fmul2_rn(ps, rr.y);
            const float2 c2 = __ffma2_rn(psy, rr.sp, make_float2(acc[u].x, acc[u].z));
            const float2 s2 = __ffma2_rn(ps, rr.cs, make_float2(acc[u].y, acc[u].w));
            acc[u] = make_float4(c2.x, s2.x, c2.y, s2.y);
        }
    }
}

// The estimate r of block q goes out (or the update built from it, with an epilogue): one 16-byte
// store where alignment allows, element by element on the ragged last block.
__device__ __forceinline__ void emit_block(const ReconstructArgs &a, uint64_t q, uint64_t q_begin, float4 r) {
    const int64_t off = (int64_t)((q - q_begin) << 2);        // offset into out
    const int64_t k = (int64_t)(q << 2);
    const float step = a.epi.base ? (a.epi.step_dev ? a.epi.step_scale * __ldg(a.epi.step_dev) : a.epi.step) : 0.f;
    if (a.vec_ok && k + 4 <= a.k_end) {
        float4 v = r;
        if (a.epi.base) {
            const float4 b = *reinterpret_cast<const float4 *>(a.epi.base + off);
            v = make_float4(fmaf(-step, r.x, b.x), fmaf(-step, r.y, b.y),
                            fmaf(-step, r.z, b.z), fmaf(-step, r.w, b.w));
            if (a.epi.shift_dst) {
                const float4 s = *reinterpret_cast<const float4 *>(a.epi.shift_src + off);
                *reinterpret_cast<float4 *>(a.epi.shift_dst + off) = s;
            }
        }
        *reinterpret_cast<float4 *>(a.out + off) = v;
    } else {
        const float vals[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int l = 0; l < 4; ++l) {
            if (k + l >= a.k_end) continue;
            float v = vals[l];
            if (a.epi.base) {
                v = fmaf(-step, v, a.epi.base[off + l]);
                if (a.epi.shift_dst) a.epi.shift_dst[off + l] = a.epi.shift_src[off + l];
            }
            a.out[off + l] = v;
        }
    }
}

__global__ void __launch_bounds__(kThreads, 3)
reconstruct_kernel(const __grid_constant__ ReconstructArgs a) {
    __shared__ uint4 table[kJChunk];              // {JPart.x0, JPart.x2, JPart.w3, bits of pbar[j]}
    const int tid = threadIdx.x;
    const uint64_t q_begin = (uint64_t)a.k_begin >> 2;
    const uint64_t q_end = ((uint64_t)a.k_end + 3) >> 2;
    const uint64_t groups = (q_end - q_begin + kGroupQ - 1) / kGroupQ;
    const float inv_m = 1.0f / (float)a.m;

    bool have_table = false;
    uint32_t table_qhi = 0;

    for (uint64_t grp = blockIdx.x; grp < groups; grp += gridDim.x) {
        // q_begin is a multiple of kGroupQ (launch_reconstruct checks), so a group never
        // straddles a multiple of 2^32 and all its blocks share the high counter word.
        const uint64_t gq0 = q_begin + grp * kGroupQ;
        const uint32_t grp_qhi = (uint32_t)(gq0 >> 32);

        float4 acc[kRecUQ];
        QPart qp[kRecUQ];
        uint64_t qv[kRecUQ];
#pragma unroll
        for (int u = 0; u < kRecUQ; ++u) {
            qv[u] = gq0 + (uint64_t)(tid + u * kThreads);
            qp[u] = philox_qpart((uint32_t)qv[u], a.t, a.keys);
            acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        }

        for (int j0 = 0; j0 < a.m; j0 += kJChunk) {
            const int jn = min(kJChunk, a.m - j0);
            const bool rebuild = !have_table || table_qhi != grp_qhi || a.m > kJChunk;
            if (rebuild) {
                __syncthreads();                  // everyone is done with the previous table
                for (int jj = tid; jj < jn; jj += kThreads) {
                    const JPart jp = philox_jpart((uint32_t)(j0 + jj), grp_qhi, a.keys);
                    table[jj] = make_uint4(jp.x0, jp.x2, jp.w3, __float_as_uint(a.pbar[j0 + jj]));
                }
                __syncthreads();
                have_table = true;
                table_qhi = grp_qhi;
            }
            // kRecJStep vectors x kRecUQ blocks are generated together (one near-one test for all)
            int jj = 0;
            for (; jj + kRecJStep <= jn; jj += kRecJStep) rec_step<kRecJStep, kRecUQ>(table + jj, qp, a.keys, acc);
            for (; jj < jn; ++jj) rec_step<1, kRecUQ>(table + jj, qp, a.keys, acc);
        }

#pragma unroll
        for (int u = 0; u < kRecUQ; ++u) {
            if (qv[u] >= q_end) continue;
            emit_block(a, qv[u], q_begin, make_float4(acc[u].x * inv_m, acc[u].y * inv_m, acc[u].z * inv_m, acc[u].w * inv_m));
        }
    }
}

// Short vectors: the kernel above would give work to a handful of CTAs only (d = 8192 is four groups),
// so here the SLICES warp groups of a CTA share out the vectors of 256 / SLICES blocks; the partial sums
// of a block meet in shared memory and are added in ascending order of the vector ranges.  Few vectors
// get few slices (a slice wants at least four vectors to generate together).
template <int SLICES>
__global__ void __launch_bounds__(kThreads)
reconstruct_small_kernel(const __grid_constant__ ReconstructArgs a) {
    constexpr int QB = kThreads / SLICES;          // blocks per CTA
    __shared__ uint4 table[kJChunk];               // as above; m <= kJChunk here
    __shared__ float4 part[SLICES][QB];
    const int tid = threadIdx.x, ql = tid % QB, slice = tid / QB;
    const uint64_t q_begin = (uint64_t)a.k_begin >> 2;
    const uint64_t q_end = ((uint64_t)a.k_end + 3) >> 2;
    const uint64_t q0 = q_begin + (uint64_t)blockIdx.x * QB;     // multiple of 32: one high counter word per CTA
    const uint32_t q_hi = (uint32_t)(q0 >> 32);
    for (int jj = tid; jj < a.m; jj += kThreads) {
        const JPart jp = philox_jpart((uint32_t)jj, q_hi, a.keys);
        table[jj] = make_uint4(jp.x0, jp.x2, jp.w3, __float_as_uint(a.pbar[jj]));
    }
    __syncthreads();
    const uint64_t q = q0 + (uint64_t)ql;
    QPart qp[1] = {philox_qpart((uint32_t)q, a.t, a.keys)};
    float4 acc[1] = {make_float4(0.f, 0.f, 0.f, 0.f)};
    const int per = ((a.m + SLICES - 1) / SLICES + 3) & ~3;      // vectors per slice, a multiple of 4
    const int j_begin = min(slice * per, a.m), j_end = min(j_begin + per, a.m);
    int jj = j_begin;
    for (; jj + 4 <= j_end; jj += 4) rec_step<4, 1>(table + jj, qp, a.keys, acc);
    for (; jj < j_end; ++jj) rec_step<1, 1>(table + jj, qp, a.keys, acc);
    part[slice][ql] = acc[0];
    __syncthreads();
    if (slice == 0 && q < q_end) {
        float4 s = part[0][ql];
#pragma unroll
        for (int r = 1; r < SLICES; ++r) {
            const float4 p = part[r][ql];
            s = make_float4(s.x + p.x, s.y + p.y, s.z + p.z, s.w + p.w);
        }
        const float inv_m = 1.0f / (float)a.m;
        emit_block(a, q, q_begin, make_float4(s.x * inv_m, s.y * inv_m, s.z * inv_m, s.w * inv_m));
    }
}

__global__ void lookahead_kernel(const float *__restrict__ x, const float *__restrict__ x_prev, float gamma, int64_t d,
                                 float *__restrict__ y) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; k < d; k += stride)
        y[k] = fmaf(gamma, x[k] - x_prev[k], x[k]);
}

struct DebugArgs {
    uint64_t q0;
    int64_t nq;
    uint32_t j;
    uint32_t t;
    RoundKeys keys;
};

__global__ void debug_philox_kernel(const __grid_constant__ DebugArgs a, uint4 *words) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; r < a.nq; r += stride) {
        const uint64_t q = a.q0 + (uint64_t)r;
        words[r] = philox4x32_10((uint32_t)q, (uint32_t)(q >> 32), a.j, a.t, a.keys);
    }
}

// Goes through the split evaluation the round kernels use, so that path is what is checked.
__global__ void debug_gaussians_kernel(const __grid_constant__ DebugArgs a, float4 *z) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; r < a.nq; r += stride) {
        const uint64_t q = a.q0 + (uint64_t)r;
        const JPart jp = philox_jpart(a.j, (uint32_t)(q >> 32), a.keys);
        const QPart qp = philox_qpart((uint32_t)q, a.t, a.keys);
        z[r] = box_muller4(philox_combine(jp, qp, a.keys));
    }
}

__global__ void debug_box_muller_kernel(const uint4 *__restrict__ words, int64_t nb, float4 *z) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; r < nb; r += stride)
        z[r] = box_muller4(words[r]);
}

unsigned grid_for(int64_t items, int threads, int cap) {
    int64_t g = (items + threads - 1) / threads;
    if (g < 1) g = 1;
    if (g > cap) g = cap;
    return (unsigned)g;
}

}  // namespace

cudaError_t launch_reconstruct(const RoundKeys &keys, uint32_t t, const float *pbar, int32_t m,
                               int64_t k_begin, int64_t k_end, float *out, int sm_count,
                               cudaStream_t stream, const ReconstructEpilogue *epilogue) {
    if (k_end <= k_begin) return cudaSuccess;
    if (k_begin % (4 * kGroupQ) != 0) return cudaErrorInvalidValue;
    ReconstructArgs a{};
    a.pbar = pbar;
    a.out = out;
    a.k_begin = k_begin;
    a.k_end = k_end;
    a.m = m;
    uintptr_t align = reinterpret_cast<uintptr_t>(out);
    if (epilogue && epilogue->base) {
        a.epi = *epilogue;
        align |= reinterpret_cast<uintptr_t>(epilogue->base);
        if (epilogue->shift_dst)
            align |= reinterpret_cast<uintptr_t>(epilogue->shift_src) | reinterpret_cast<uintptr_t>(epilogue->shift_dst);
    }
    a.vec_ok = (align % 16) == 0 ? 1 : 0;
    a.t = t;
    a.keys = keys;
    const int64_t nq = ((k_end + 3) >> 2) - (k_begin >> 2);
    const int64_t groups = (nq + kGroupQ - 1) / kGroupQ;
    if (groups < 8 * (int64_t)sm_count && m <= kJChunk) {    // too few groups to go round evenly: smaller units
        // more slices = fewer blocks per CTA = more CTAs: as many as it takes to go round, while a slice
        // keeps at least four vectors
        int slices = 1;
        while (slices < 8 && m >= 8 * slices && nq / (kThreads / slices) < 4 * (int64_t)sm_count) slices *= 2;
        const unsigned grid = (unsigned)((nq + kThreads / slices - 1) / (kThreads / slices));
        switch (slices) {
            case 8: reconstruct_small_kernel<8><<<grid, kThreads, 0, stream>>>(a); break;
            case 4: reconstruct_small_kernel<4><<<grid, kThreads, 0, stream>>>(a); break;
            case 2: reconstruct_small_kernel<2><<<grid, kThreads, 0, stream>>>(a); break;
            default: reconstruct_small_kernel<1><<<grid, kThreads, 0, stream>>>(a); break;
        }
        return cudaGetLastError();
    }
    int64_t grid = (int64_t)sm_count * 3;     // three resident CTAs per SM (register-limited)
    if (grid > groups) grid = groups;
    reconstruct_kernel<<<(unsigned)grid, kThreads, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_lookahead(const float *x, const float *x_prev, float gamma, int64_t d, float *y,
                             cudaStream_t stream) {
    lookahead_kernel<<<grid_for(d, 256, 148 * 8), 256, 0, stream>>>(x, x_prev, gamma, d, y);
    return cudaGetLastError();
}

cudaError_t launch_debug_philox(const RoundKeys &keys, uint32_t t, uint32_t j, uint64_t q0, int64_t nq,
                                uint32_t *words, cudaStream_t stream) {
    if (nq <= 0) return cudaSuccess;
    DebugArgs a{q0, nq, j, t, keys};
    debug_philox_kernel<<<grid_for(nq, 256, 148 * 8), 256, 0, stream>>>(a, reinterpret_cast<uint4 *>(words));
    return cudaGetLastError();
}

cudaError_t launch_debug_gaussians(const RoundKeys &keys, uint32_t t, uint32_t j, uint64_t q0, int64_t nq,
                                   float *z, cudaStream_t stream) {
    if (nq <= 0) return cudaSuccess;
    DebugArgs a{q0, nq, j, t, keys};
    debug_gaussians_kernel<<<grid_for(nq, 256, 148 * 8), 256, 0, stream>>>(a, reinterpret_cast<float4 *>(z));
    return cudaGetLastError();
}

cudaError_t launch_debug_box_muller(const uint32_t *words, int64_t nb, float *z, cudaStream_t stream) {
    if (nb <= 0) return cudaSuccess;
    debug_box_muller_kernel<<<grid_for(nb, 256, 148 * 8), 256, 0, stream>>>(
        reinterpret_cast<const uint4 *>(words), nb, reinterpret_cast<float4 *>(z));
    return cudaGetLastError();
}

}  // namespace core
