// Projection for 9..16 machines with the multiply-adds on the tensor cores.
//
// With many machines the fp32 multiply-adds (four per machine and Gaussian) cost more issue slots
// than generating the Gaussians.  Here a warp treats one step as a small matrix product
//     D[16 machines x 8 vectors] += A[16 machines x 8 coordinates] * B[8 coordinates x 8 vectors]
// (mma.sync m16n8k8, tf32 inputs, fp32 accumulate).  Lane (g, t) = (lane / 4, lane % 4) generates the
// four Gaussians of vector g and coordinate block t of the step, which are exactly the B entries the
// instruction expects from that lane; the A entries come from the shared-memory gradient tile.
// tf32 keeps 10 mantissa bits, far too few for the 1e-4 ||g|| bound, so every operand is split into a
// tf32 head and a tail (x = hi + lo, both exact in fp32) and the three products hi*hi, lo*hi, hi*lo are
// accumulated (relative error about 2^-21 per product).  bf16 gradients are exact in tf32: no tail.
// The partial sums leave the kernel in the same layout as those of the scalar kernel.
#include "core_internal.h"

#include <cuda_bf16.h>

namespace core {

namespace {

constexpr int kMmaJT = 2;                 // vector groups (of 8) per warp
constexpr int kMmaVecPerCta = 8 * 8 * kMmaJT;   // 8 warps x 8 vectors x JT

struct MmaArgs {
    const void *G;
    int64_t ldg;
    int64_t d;
    int64_t tiles;
    uint64_t q_base;
    float *partial;
    int n;
    int m;
    int aligned;
    uint32_t t;
    RoundKeys keys;
};

__device__ __forceinline__ float tf32_head(float x) { return __uint_as_float(__float_as_uint(x) & 0xFFFFE000u); }

__device__ __forceinline__ void mma_tf32(float (&c)[4], const float (&a)[4], float b0, float b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(__float_as_uint(a[0])), "r"(__float_as_uint(a[1])), "r"(__float_as_uint(a[2])),
          "r"(__float_as_uint(a[3])), "r"(__float_as_uint(b0)), "r"(__float_as_uint(b1)));
}

// TILE_Q coordinate blocks per tile; rows of the tile are padded by four float4 so that the eight
// machines a quarter-warp reads fall into different banks.
template <int TILE_Q, typename GT>
__global__ void __launch_bounds__(kThreads, 2)
project_mma_kernel(const __grid_constant__ MmaArgs a) {
    constexpr bool BF16 = sizeof(GT) == 2;
    constexpr bool SPLIT_A = !BF16;
    constexpr int TILE = 4 * TILE_Q;
    constexpr int RS = TILE_Q + 4;                                  // row stride in float4
    constexpr int PLANE = 16 * RS;                                  // float4 per (hi or lo) tile
    constexpr int STAGE = PLANE * (SPLIT_A ? 2 : 1);                // float4 per stage
    constexpr int PIECES = 16 * TILE_Q / (BF16 ? 2 : 1);            // 16-byte pieces of input per tile
    constexpr int PPT = PIECES / kThreads;
    static_assert(PIECES % kThreads == 0, "tile must split evenly over the CTA");

    extern __shared__ __align__(16) unsigned char smem_raw[];
    float4 *stage0 = reinterpret_cast<float4 *>(smem_raw);
    float4 *stage1 = stage0 + STAGE;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t4 = lane & 3;
    const GT *G = static_cast<const GT *>(a.G);
    const int jbase = blockIdx.y * kMmaVecPerCta + warp * 8 * kMmaJT;     // first vector of this warp

    const int64_t per = (a.tiles + gridDim.x - 1) / gridDim.x;
    const int64_t tile_begin = (int64_t)blockIdx.x * per;
    const int64_t tile_end = min(tile_begin + per, a.tiles);

    float outer[kMmaJT][4];
#pragma unroll
    for (int v = 0; v < kMmaJT; ++v)
#pragma unroll
        for (int c = 0; c < 4; ++c) outer[v][c] = 0.f;

    uint4 held[PPT];
    auto tile_is_fast = [&](int64_t tile) { return a.aligned && (tile + 1) * TILE <= a.d; };

    auto begin_stage = [&](int64_t tile) {
        if (!tile_is_fast(tile)) return;
        const int64_t k0 = tile * TILE;
#pragma unroll
        for (int r = 0; r < PPT; ++r) {
            const int piece = tid + r * kThreads;
            constexpr int PER_ROW = PIECES / 16;
            const int i = piece / PER_ROW, c = piece % PER_ROW;
            const int64_t off = (int64_t)i * a.ldg + k0 + (BF16 ? 8 : 4) * c;
            held[r] = (i < a.n) ? __ldg(reinterpret_cast<const uint4 *>(G + off)) : make_uint4(0, 0, 0, 0);
        }
    };

    auto store_block = [&](float4 *stage, int i, int q, float4 v) {
        if constexpr (SPLIT_A) {
            const float4 hi = make_float4(tf32_head(v.x), tf32_head(v.y), tf32_head(v.z), tf32_head(v.w));
            stage[i * RS + q] = hi;
            stage[PLANE + i * RS + q] = make_float4(v.x - hi.x, v.y - hi.y, v.z - hi.z, v.w - hi.w);
        } else {
            stage[i * RS + q] = v;
        }
    };

    auto finish_stage = [&](int64_t tile, float4 *stage) {
        if (tile_is_fast(tile)) {
#pragma unroll
            for (int r = 0; r < PPT; ++r) {
                const int piece = tid + r * kThreads;
                constexpr int PER_ROW = PIECES / 16;
                const int i = piece / PER_ROW, c = piece % PER_ROW;
                const uint4 h = held[r];
                if constexpr (BF16) {
                    store_block(stage, i, 2 * c, make_float4(__uint_as_float(h.x << 16), __uint_as_float(h.x & 0xFFFF0000u),
                                                            __uint_as_float(h.y << 16), __uint_as_float(h.y & 0xFFFF0000u)));
                    store_block(stage, i, 2 * c + 1, make_float4(__uint_as_float(h.z << 16), __uint_as_float(h.z & 0xFFFF0000u),
                                                                __uint_as_float(h.w << 16), __uint_as_float(h.w & 0xFFFF0000u)));
                } else {
                    store_block(stage, i, c, make_float4(__uint_as_float(h.x), __uint_as_float(h.y), __uint_as_float(h.z),
                                                         __uint_as_float(h.w)));
                }
            }
            return;
        }
        // ragged or unaligned tile: element by element, zero beyond d and beyond n
        const int64_t k0 = tile * TILE;
        for (int e = tid; e < 16 * TILE_Q; e += kThreads) {
            const int i = e / TILE_Q, q = e % TILE_Q;
            float vals[4] = {0.f, 0.f, 0.f, 0.f};
            if (i < a.n) {
#pragma unroll
                for (int l = 0; l < 4; ++l) {
                    const int64_t k = k0 + 4 * q + l;
                    if (k < a.d) {
                        if constexpr (BF16)
                            vals[l] = __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short *>(G) +
                                                                      (int64_t)i * a.ldg + k) << 16);
                        else
                            vals[l] = __ldg(reinterpret_cast<const float *>(G) + (int64_t)i * a.ldg + k);
                    }
                }
            }
            store_block(stage, i, q, make_float4(vals[0], vals[1], vals[2], vals[3]));
        }
    };

    if (tile_begin < tile_end) {
        begin_stage(tile_begin);
        finish_stage(tile_begin, stage0);
    }
    __syncthreads();

    for (int64_t tile = tile_begin; tile < tile_end; ++tile) {
        float4 *cur = ((tile - tile_begin) & 1) ? stage1 : stage0;
        float4 *nxt = ((tile - tile_begin) & 1) ? stage0 : stage1;
        const bool more = tile + 1 < tile_end;
        if (more) begin_stage(tile + 1);

        const uint64_t q0 = a.q_base + (uint64_t)tile * TILE_Q;
        const uint32_t q0_lo = (uint32_t)q0, q_hi = (uint32_t)(q0 >> 32);
        JPart jp[kMmaJT];
#pragma unroll
        for (int v = 0; v < kMmaJT; ++v) jp[v] = philox_jpart((uint32_t)(jbase + v * 8 + g), q_hi, a.keys);

        float acc[kMmaJT][4];
#pragma unroll
        for (int v = 0; v < kMmaJT; ++v)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[v][c] = 0.f;

        for (int qs = 0; qs < TILE_Q; qs += 4) {
            const int q = qs + t4;                                   // this lane's block in the step
            const QPart qp = philox_qpart(q0_lo + (uint32_t)q, a.t, a.keys);
            uint4 w[kMmaJT];
#pragma unroll
            for (int v = 0; v < kMmaJT; ++v) w[v] = philox_combine(jp[v], qp, a.keys);
            float4 z[kMmaJT];
            box_muller4xN<kMmaJT>(w, z);

            const float4 row_g = cur[g * RS + q];                    // machine g, block q (tf32 heads)
            const float4 row_g8 = cur[(g + 8) * RS + q];             // machine g + 8
            // fragment order of the instruction: (row g, k t), (row g+8, k t), (row g, k t+4), (row g+8, k t+4)
            const float ahi[2][4] = {{row_g.x, row_g8.x, row_g.y, row_g8.y},
                                     {row_g.z, row_g8.z, row_g.w, row_g8.w}};
            float alo[2][4];
            if constexpr (SPLIT_A) {
                const float4 t_lo = cur[PLANE + g * RS + q];
                const float4 t_hi = cur[PLANE + (g + 8) * RS + q];
                alo[0][0] = t_lo.x; alo[0][1] = t_hi.x; alo[0][2] = t_lo.y; alo[0][3] = t_hi.y;
                alo[1][0] = t_lo.z; alo[1][1] = t_hi.z; alo[1][2] = t_lo.w; alo[1][3] = t_hi.w;
            }
#pragma unroll
            for (int v = 0; v < kMmaJT; ++v) {
                const float zz[4] = {z[v].x, z[v].y, z[v].z, z[v].w};
#pragma unroll
                for (int s = 0; s < 2; ++s) {                        // coordinates (2s, 2s+1) of the blocks
                    const float b0 = zz[2 * s], b1 = zz[2 * s + 1];
                    const float b0h = tf32_head(b0), b1h = tf32_head(b1);
                    mma_tf32(acc[v], ahi[s], b0h, b1h);
                    mma_tf32(acc[v], ahi[s], b0 - b0h, b1 - b1h);
                    if constexpr (SPLIT_A) mma_tf32(acc[v], alo[s], b0h, b1h);
                }
            }
        }
#pragma unroll
        for (int v = 0; v < kMmaJT; ++v)
#pragma unroll
            for (int c = 0; c < 4; ++c) outer[v][c] += acc[v][c];

        if (more) finish_stage(tile + 1, nxt);
        __syncthreads();
    }

    // lane (g, t4) holds machines {g, g+8} x vectors {2 t4, 2 t4 + 1} of each of its groups
#pragma unroll
    for (int v = 0; v < kMmaJT; ++v) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int i = g + 8 * (c >> 1);
            const int j = jbase + v * 8 + 2 * t4 + (c & 1);
            if (i < a.n && j < a.m) a.partial[((int64_t)blockIdx.x * a.n + i) * a.m + j] = outer[v][c];
        }
    }
}

}  // namespace

bool project_mma_applies(int32_t n_group, int32_t m) { return n_group > 8 && m >= 64; }

void fill_project_mma_plan(ProjectPlan &p, int32_t m, int64_t d, int dtype, int sm_count) {
    p.mma = 1;
    p.nb = 16;
    p.jt = kMmaJT;
    p.uq = 1;
    p.tile_q = dtype == 1 ? 128 : 64;
    p.tj = 64;                         // reporting only: 8 warps x 8 vectors
    p.tq = 4;
    p.grid_y = (m + kMmaVecPerCta - 1) / kMmaVecPerCta;
    p.tiles = (d + 4 * (int64_t)p.tile_q - 1) / (4 * (int64_t)p.tile_q);
    const size_t plane = (size_t)16 * (p.tile_q + 4) * 16;
    p.smem = 2 * plane * (dtype == 1 ? 1 : 2);
    int64_t gx = (int64_t)sm_count * 2 / p.grid_y;
    if (gx < 1) gx = 1;
    if (gx > p.tiles) gx = p.tiles;
    p.grid_x = (int)gx;
}

cudaError_t launch_project_mma(const ProjectPlan &plan, const RoundKeys &keys, uint32_t t, const void *G, int dtype,
                               int32_t n, int64_t ldg, int64_t d, int32_t m, uint64_t q_base, float *partial,
                               cudaStream_t stream) {
    MmaArgs a{};
    a.G = G;
    a.ldg = ldg;
    a.d = d;
    a.tiles = plan.tiles;
    a.q_base = q_base;
    a.partial = partial;
    a.n = n;
    a.m = m;
    const size_t es = dtype == 1 ? 2 : 4;
    a.aligned = ((reinterpret_cast<uintptr_t>(G) % 16) == 0 && ((size_t)ldg * es) % 16 == 0) ? 1 : 0;
    a.t = t;
    a.keys = keys;
    dim3 grid(plan.grid_x, plan.grid_y);
    auto go = [&](auto kernel) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem);
        if (e != cudaSuccess) return e;
        kernel<<<grid, kThreads, plan.smem, stream>>>(a);
        return cudaGetLastError();
    };
    if (dtype == 1) return go(project_mma_kernel<128, __nv_bfloat16>);
    return go(project_mma_kernel<64, float>);
}

}  // namespace core
