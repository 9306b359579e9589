// Fused generate-and-project kernel: P[i][j] = <g_i, xi_j> (Algorithm 1, sender's step;
// Algorithm 2, "machine i sends p_ij"), for up to 16 machines per pass.
//
// The common vectors xi_j are generated in registers and never stored.  A CTA owns a
// contiguous range of coordinate tiles and a range of vectors.  Thread (jl, ql) keeps JT
// (4, or 2 with 16 machines) vectors j = jbase + jl + v*tj fixed and walks the coordinate blocks ql*UQ, ql*UQ + tq*UQ, ...
// of every tile: one Philox counter gives the four Gaussians of (block, vector), which
// meet the NB machine gradients of that block read (as broadcasts) from shared memory.
// The gradient tile is staged once per CTA and tile, so G is read from HBM once per
// vector group.  Sums are kept in two levels (per tile, then across tiles) to bound the
// fp32 chain length, reduced across the ql lanes in a fixed order, and written as one
// partial P per CTA column; a second kernel adds the columns in ascending order.
#include "core_internal.h"

#include <cuda_bf16.h>

namespace core {

namespace {

__host__ __device__ constexpr int tile_q_for(int nb) { return nb <= 2 ? 1024 : 2048 / nb; }
// Short vectors: with the tile above only a handful of CTAs would get work (d = 8192 is 8 tiles for
// 8 machines), so small problems are cut into tiles of 32 blocks instead.
constexpr int kSmallTileQ = 32;
// In between, and for few vectors (a tile of 32 blocks keeps at least 8 threads across the vectors, which
// idle when there are fewer than 8 x JT of them): tiles of 128 blocks.
constexpr int kMediumTileQ = 128;

struct ProjectArgs {
    const void *G;
    int64_t ldg;
    int64_t d;
    int64_t tiles;
    uint64_t q_base;
    float *partial;
    int n;
    int m;
    int tj;          // threads across vectors
    int tj_log2;
    int aligned;     // rows may be copied in 16-byte pieces
    int splits;      // > 0: row i is the sum of `splits` arrays ldg apart, times `scale` (see launch_project)
    float scale;
    uint32_t t;
    RoundKeys keys;
};

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src, bool valid) {
    unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
    int bytes = valid ? 16 : 0;   // zero bytes read: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(gmem_src), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
}

__device__ __forceinline__ float load_elem(const float *p) { return __ldg(p); }
__device__ __forceinline__ float load_elem(const __nv_bfloat16 *p) {
    return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short *>(p)) << 16);
}

template <int NB, int JT, int UQ, int TILE_Q, typename GT>
__global__ void __launch_bounds__(kThreads, 2)
project_kernel(const __grid_constant__ ProjectArgs a) {
    constexpr int TILE = 4 * TILE_Q;
    constexpr bool BF16 = sizeof(GT) == 2;
    constexpr int PIECES = NB * TILE_Q / (BF16 ? 2 : 1);          // 16-byte pieces per tile
    constexpr int PIECES_PER_THREAD = (PIECES + kThreads - 1) / kThreads;
    constexpr bool EVEN = PIECES % kThreads == 0;                 // otherwise the last round is partial

    extern __shared__ __align__(16) unsigned char smem_raw[];
    float4 *stage0 = reinterpret_cast<float4 *>(smem_raw);
    float4 *stage1 = stage0 + NB * TILE_Q;
    // the block-dependent half of Philox for every block of a tile, tabulated once per CTA and tile
    // ({hi_b, lo_b, w3, -}; double buffered like the gradient tile) instead of once per thread and step
    uint4 *qtab0 = reinterpret_cast<uint4 *>(stage1 + NB * TILE_Q);
    uint4 *qtab1 = qtab0 + TILE_Q;

    const int tid = threadIdx.x;
    const int tj = a.tj;
    const int tq = kThreads >> a.tj_log2;
    const int jl = tid & (tj - 1);
    const int ql = tid >> a.tj_log2;
    const int jbase = blockIdx.y * tj * JT;
    const GT *G = static_cast<const GT *>(a.G);

    // this CTA's tiles
    const int64_t per = (a.tiles + gridDim.x - 1) / gridDim.x;
    const int64_t tile_begin = (int64_t)blockIdx.x * per;
    const int64_t tile_end = min(tile_begin + per, a.tiles);

    float outer[NB][JT];
#pragma unroll
    for (int i = 0; i < NB; ++i)
#pragma unroll
        for (int v = 0; v < JT; ++v) outer[i][v] = 0.f;

    uint4 held[BF16 ? PIECES_PER_THREAD : 1];   // bf16 path: next tile's pieces in flight

    // Fast staging needs whole 16-byte pieces inside every row.
    auto tile_is_fast = [&](int64_t tile) { return a.aligned && (tile + 1) * TILE <= a.d; };

    // Start moving tile -> stage.  fp32: asynchronous copies straight to shared memory.
    // bf16: loads into registers, converted and stored by finish_stage().
    auto begin_stage = [&](int64_t tile, float4 *stage) {
        if (!tile_is_fast(tile)) return;
        const int64_t k0 = tile * TILE;
#pragma unroll
        for (int r = 0; r < PIECES_PER_THREAD; ++r) {
            const int piece = tid + r * kThreads;
            if (!EVEN && piece >= PIECES) break;
            if constexpr (BF16) {
                const int i = piece / (TILE_Q / 2);
                const int c = piece % (TILE_Q / 2);
                held[r] = (i < a.n) ? __ldg(reinterpret_cast<const uint4 *>(G + (int64_t)i * a.ldg + k0 + 8 * c))
                                    : make_uint4(0, 0, 0, 0);
            } else {
                const int i = piece / TILE_Q;
                const int c = piece % TILE_Q;
                const bool valid = i < a.n;
                const GT *src = G + (valid ? (int64_t)i * a.ldg : 0) + k0 + 4 * c;
                cp_async16(stage + piece, src, valid);
            }
        }
    };

    auto finish_stage = [&](int64_t tile, float4 *stage) {
        if (tile_is_fast(tile)) {
            if constexpr (BF16) {
#pragma unroll
                for (int r = 0; r < PIECES_PER_THREAD; ++r) {
                    const int piece = tid + r * kThreads;
                    if (!EVEN && piece >= PIECES) break;
                    const uint4 h = held[r];
                    // a bf16 is the upper half of an fp32
                    stage[2 * piece] = make_float4(__uint_as_float(h.x << 16), __uint_as_float(h.x & 0xFFFF0000u),
                                                   __uint_as_float(h.y << 16), __uint_as_float(h.y & 0xFFFF0000u));
                    stage[2 * piece + 1] = make_float4(__uint_as_float(h.z << 16), __uint_as_float(h.z & 0xFFFF0000u),
                                                       __uint_as_float(h.w << 16), __uint_as_float(h.w & 0xFFFF0000u));
                }
            }
            return;
        }
        float *flat = reinterpret_cast<float *>(stage);
        const int64_t k0 = tile * TILE;
        if constexpr (!BF16) {
            if (a.splits > 0) {
                // summed rows (d and ldg are multiples of 4 here): one block of four coordinates per thread
                // step, the `splits` 16-byte loads of a block independent of one another
                for (int e = tid; e < NB * TILE_Q; e += kThreads) {
                    const int i = e / TILE_Q;
                    const int64_t k = k0 + 4 * (e % TILE_Q);
                    float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (i < a.n && k < a.d) {
                        const float4 *src = reinterpret_cast<const float4 *>(G + (int64_t)i * a.splits * a.ldg + k);
                        const int64_t stride4 = a.ldg >> 2;
#pragma unroll 6
                        for (int c = 0; c < a.splits; ++c) {
                            const float4 v = __ldg(src + (int64_t)c * stride4);
                            sum = make_float4(sum.x + v.x, sum.y + v.y, sum.z + v.z, sum.w + v.w);
                        }
                        sum = make_float4(sum.x * a.scale, sum.y * a.scale, sum.z * a.scale, sum.w * a.scale);
                    }
                    stage[e] = sum;
                }
                return;
            }
        }
        // ragged or unaligned tile: element by element, zero beyond d and beyond n
        for (int e = tid; e < NB * TILE; e += kThreads) {
            const int i = e / TILE;
            const int64_t k = k0 + (e % TILE);
            float val = 0.f;
            if (i < a.n && k < a.d) val = load_elem(G + (int64_t)i * a.ldg + k);
            flat[e] = val;
        }
    };

    auto fill_qtab = [&](int64_t tile, uint4 *tab) {
        const uint32_t first = (uint32_t)(a.q_base + (uint64_t)tile * TILE_Q);
        for (int e = tid; e < TILE_Q; e += kThreads) {
            const QPart qp = philox_qpart(first + (uint32_t)e, a.t, a.keys);
            tab[e] = make_uint4(qp.hi_b, qp.lo_b, qp.w3, 0u);
        }
    };

    if (tile_begin < tile_end) {
        begin_stage(tile_begin, stage0);
        fill_qtab(tile_begin, qtab0);
        finish_stage(tile_begin, stage0);
    }
    cp_async_wait_all();
    __syncthreads();

    // the vector-dependent half of Philox changes only with the high word of the block index
    JPart jp[JT];
    uint32_t jp_q_hi = 0;
    bool have_jp = false;

    for (int64_t tile = tile_begin; tile < tile_end; ++tile) {
        float4 *cur = ((tile - tile_begin) & 1) ? stage1 : stage0;
        float4 *nxt = ((tile - tile_begin) & 1) ? stage0 : stage1;
        const uint4 *qtab = ((tile - tile_begin) & 1) ? qtab1 : qtab0;
        const bool more = tile + 1 < tile_end;
        if (more) {
            begin_stage(tile + 1, nxt);
            fill_qtab(tile + 1, ((tile - tile_begin) & 1) ? qtab0 : qtab1);
        }

        const uint64_t q0 = a.q_base + (uint64_t)tile * TILE_Q;   // multiple of TILE_Q: no carry inside
        const uint32_t q_hi = (uint32_t)(q0 >> 32);
        if (!have_jp || q_hi != jp_q_hi) {
#pragma unroll
            for (int v = 0; v < JT; ++v) jp[v] = philox_jpart((uint32_t)(jbase + jl + v * tj), q_hi, a.keys);
            jp_q_hi = q_hi;
            have_jp = true;
        }

        float acc[NB][JT];
#pragma unroll
        for (int i = 0; i < NB; ++i)
#pragma unroll
            for (int v = 0; v < JT; ++v) acc[i][v] = 0.f;

        for (int qq = ql * UQ; qq < TILE_Q; qq += tq * UQ) {
            uint4 w[UQ * JT];
#pragma unroll
            for (int u = 0; u < UQ; ++u) {
                const uint4 e = qtab[qq + u];
                QPart qp;
                qp.hi_b = e.x;
                qp.lo_b = e.y;
                qp.w3 = e.z;
#pragma unroll
                for (int v = 0; v < JT; ++v) w[u * JT + v] = philox_combine(jp[v], qp, a.keys);
            }
            float4 z[UQ * JT];
            box_muller4xN<UQ * JT>(w, z);
#pragma unroll
            for (int i = 0; i < NB; ++i) {
#pragma unroll
                for (int u = 0; u < UQ; ++u) {
                    const float4 g = cur[i * TILE_Q + qq + u];
#pragma unroll
                    for (int v = 0; v < JT; ++v) {
                        const float4 zz = z[u * JT + v];
                        float s = acc[i][v];
                        s = fmaf(g.x, zz.x, s);
                        s = fmaf(g.y, zz.y, s);
                        s = fmaf(g.z, zz.z, s);
                        s = fmaf(g.w, zz.w, s);
                        acc[i][v] = s;
                    }
                }
            }
        }
#pragma unroll
        for (int i = 0; i < NB; ++i)
#pragma unroll
            for (int v = 0; v < JT; ++v) outer[i][v] += acc[i][v];

        if (more) finish_stage(tile + 1, nxt);
        cp_async_wait_all();
        __syncthreads();
    }

    // fixed-order reduction over the ql lanes
    float *red = reinterpret_cast<float *>(smem_raw);
    const int plane = NB * JT * tj;
#pragma unroll
    for (int i = 0; i < NB; ++i)
#pragma unroll
        for (int v = 0; v < JT; ++v) red[ql * plane + (i * JT + v) * tj + jl] = outer[i][v];
    __syncthreads();
    for (int idx = tid; idx < plane; idx += kThreads) {
        float s = 0.f;
        for (int l = 0; l < tq; ++l) s += red[l * plane + idx];
        const int lane = idx & (tj - 1);
        const int iv = idx >> a.tj_log2;
        const int i = iv / JT, v = iv % JT;
        const int j = jbase + lane + v * tj;
        if (i < a.n && j < a.m) a.partial[((int64_t)blockIdx.x * a.n + i) * a.m + j] = s;
    }
}

template <int NB, int JT, int UQ, int TILE_Q>
cudaError_t launch_tiled(const ProjectPlan &plan, const ProjectArgs &args, int dtype, cudaStream_t stream) {
    dim3 grid(plan.grid_x, plan.grid_y);
    auto go = [&](auto kernel) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem);
        if (e != cudaSuccess) return e;
        kernel<<<grid, kThreads, plan.smem, stream>>>(args);
        return cudaGetLastError();
    };
    if (dtype == 1) return go(project_kernel<NB, JT, UQ, TILE_Q, __nv_bfloat16>);
    return go(project_kernel<NB, JT, UQ, TILE_Q, float>);
}

template <int NB, int JT, int UQ>
cudaError_t launch_typed(const ProjectPlan &plan, const ProjectArgs &args, int dtype, cudaStream_t stream) {
    if (plan.tile_q == kSmallTileQ) return launch_tiled<NB, JT, UQ, kSmallTileQ>(plan, args, dtype, stream);
    if (plan.tile_q == kMediumTileQ && kMediumTileQ != tile_q_for(NB))
        return launch_tiled<NB, JT, UQ, kMediumTileQ>(plan, args, dtype, stream);
    return launch_tiled<NB, JT, UQ, tile_q_for(NB)>(plan, args, dtype, stream);
}

__global__ void finish_project_kernel(const float *__restrict__ partial, int chunks, int n, int m,
                                      float *__restrict__ P, int accumulate) {
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t total = (int64_t)n * m;
    if (idx >= total) return;
    float s = accumulate ? P[idx] : 0.f;
    for (int c = 0; c < chunks; ++c) s += partial[(int64_t)c * total + idx];
    P[idx] = s;
}

__global__ void aggregate_kernel(const float *__restrict__ P, int n, int m, float *__restrict__ pbar) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= m) return;
    float s = 0.f;
    for (int i = 0; i < n; ++i) s += P[(int64_t)i * m + j];
    pbar[j] = s / (float)n;
}

// Both of the above in one launch for a single group of machines whose messages nobody asks for:
// the same sums in the same order, so pbar is bitwise what the two kernels give.
__global__ void finish_aggregate_kernel(const float *__restrict__ partial, int chunks, int n, int m,
                                        float *__restrict__ pbar) {
    __shared__ float message[kMaxGroupTc][32];     // P[i][j] of this block's 32 vectors
    const int j = blockIdx.x * 32 + threadIdx.x;
    const int64_t total = (int64_t)n * m;
    for (int i = threadIdx.y; i < n; i += blockDim.y) {
        float p = 0.f;
        if (j < m)
            for (int c = 0; c < chunks; ++c) p += partial[(int64_t)c * total + (int64_t)i * m + j];
        message[i][threadIdx.x] = p;
    }
    __syncthreads();
    if (threadIdx.y != 0 || j >= m) return;
    float s = 0.f;
    for (int r = 0; r < n; ++r) s += message[r][threadIdx.x];
    pbar[j] = s / (float)n;
}

int ilog2(int x) {
    int l = 0;
    while ((1 << l) < x) ++l;
    return l;
}

}  // namespace

namespace {
int g_force_kernel = -1;
}

void project_force_kernel(int kind) { g_force_kernel = kind; }

int32_t project_group(int32_t n_left, int32_t m) {
    if (n_left > kMaxGroup && g_force_kernel != 0 && g_force_kernel != 1) {
        const int32_t most = project_tc_max_group(m);
        const int32_t wide = n_left < most ? n_left : most;
        if (g_force_kernel == 2 || project_tc_applies(wide, m)) return wide;
    }
    return n_left < kMaxGroup ? n_left : kMaxGroup;
}

ProjectPlan make_project_plan(int32_t n_group, int32_t m, int64_t d, int dtype, int sm_count) {
    ProjectPlan p{};
    const bool tc = g_force_kernel == 2 ? n_group <= project_tc_max_group(m) : (g_force_kernel < 0 && project_tc_applies(n_group, m));
    if (tc) {
        fill_project_tc_plan(p, n_group, m, d, dtype, sm_count);
        return p;
    }
    if (g_force_kernel != 0 && n_group <= kMaxGroup && project_mma_applies(n_group, m)) {
        fill_project_mma_plan(p, m, d, dtype, sm_count);
        return p;
    }
    p.nb = 1;
    while (p.nb < n_group) p.nb *= 2;
    // four generator calls per thread step: 4 vectors x 1 block (fewer machines) or 2 x 1
    p.jt = (p.nb >= 8) ? 2 : 4;
    p.uq = (p.nb == 8) ? 2 : 1;
    p.tile_q = tile_q_for(p.nb);
    {
        // would the large tiles leave SMs without a CTA, or give the CTAs too few tiles to share out evenly?
        const int tj_big = m >= kThreads * p.jt ? kThreads : 0;   // grid_y > 1 only then
        const int64_t gy = tj_big ? (m + kThreads * p.jt - 1) / (kThreads * p.jt) : 1;
        const int64_t tiles_big = (d + 4 * (int64_t)p.tile_q - 1) / (4 * (int64_t)p.tile_q);
        if (tiles_big * gy < 8 * (int64_t)sm_count) {
            int tj_want = 1;
            while (tj_want < (m + p.jt - 1) / p.jt && tj_want < kThreads) tj_want *= 2;
            const bool small_fits = kThreads * p.uq / kSmallTileQ <= tj_want;      // no idle threads across vectors
            const int64_t tiles_medium = (d + 4 * (int64_t)kMediumTileQ - 1) / (4 * (int64_t)kMediumTileQ);
            const bool medium_fills = tiles_medium * gy >= sm_count / 2;
            p.tile_q = (small_fits || !medium_fills || kMediumTileQ > p.tile_q) ? kSmallTileQ : kMediumTileQ;
        }
    }
    int want = (m + p.jt - 1) / p.jt;                 // threads needed across vectors
    int tj = 1;
    while (tj < want && tj < kThreads) tj *= 2;
    const int min_tj = kThreads * p.uq / p.tile_q;    // keeps tq * uq <= tile_q
    if (tj < min_tj) tj = min_tj;
    p.tj = tj;
    p.tq = kThreads / tj;
    p.grid_y = (m + tj * p.jt - 1) / (tj * p.jt);
    p.tiles = (d + 4 * (int64_t)p.tile_q - 1) / (4 * (int64_t)p.tile_q);
    const size_t stage = (size_t)p.nb * p.tile_q * 16;
    const size_t red = (size_t)kThreads * p.nb * p.jt * 4;
    const size_t tiles_and_tables = 2 * stage + 2 * (size_t)p.tile_q * 16;   // two gradient tiles + two Philox block tables
    p.smem = tiles_and_tables > red ? tiles_and_tables : red;
    int ctas_per_sm = (int)((size_t)(200 * 1024) / p.smem);
    if (ctas_per_sm > 2) ctas_per_sm = 2;
    if (ctas_per_sm < 1) ctas_per_sm = 1;
    int64_t gx = (int64_t)sm_count * ctas_per_sm / p.grid_y;
    if (gx < 1) gx = 1;
    if (gx > p.tiles) gx = p.tiles;
    p.grid_x = (int)gx;
    (void)dtype;
    return p;
}

cudaError_t launch_project(const ProjectPlan &plan, const RoundKeys &keys, uint32_t t, const void *G,
                           int dtype, int32_t n, int64_t ldg, int64_t d, int32_t m, uint64_t q_base,
                           float *partial, cudaStream_t stream, int splits, float scale) {
    if (splits > 0 && (plan.mma != 0 || dtype != 0 || d % 4 != 0 || ldg % 4 != 0 ||
                       reinterpret_cast<uintptr_t>(G) % 16 != 0))
        return cudaErrorInvalidValue;
    if (plan.mma == 2) return launch_project_tc(plan, keys, t, G, dtype, n, ldg, d, m, q_base, partial, stream);
    if (plan.mma == 1) return launch_project_mma(plan, keys, t, G, dtype, n, ldg, d, m, q_base, partial, stream);
    ProjectArgs a{};
    a.G = G;
    a.ldg = ldg;
    a.d = d;
    a.tiles = plan.tiles;
    a.q_base = q_base;
    a.partial = partial;
    a.n = n;
    a.m = m;
    a.tj = plan.tj;
    a.tj_log2 = ilog2(plan.tj);
    const size_t es = dtype == 1 ? 2 : 4;
    a.aligned = ((reinterpret_cast<uintptr_t>(G) % 16) == 0 && ((size_t)ldg * es) % 16 == 0) ? 1 : 0;
    a.splits = splits;
    a.scale = scale;
    if (splits > 0) a.aligned = 0;      // summed rows are formed element by element while the tile is staged
    a.t = t;
    a.keys = keys;
    switch (plan.nb) {
        case 1: return launch_typed<1, 4, 1>(plan, a, dtype, stream);
        case 2: return launch_typed<2, 4, 1>(plan, a, dtype, stream);
        case 4: return launch_typed<4, 4, 1>(plan, a, dtype, stream);
        case 8: return launch_typed<8, 2, 2>(plan, a, dtype, stream);
        default: return launch_typed<16, 2, 1>(plan, a, dtype, stream);
    }
}

cudaError_t launch_finish_project(const float *partial, int chunks, int32_t n, int32_t m, float *P,
                                  bool accumulate, cudaStream_t stream) {
    const int64_t total = (int64_t)n * m;
    const int threads = 128;
    finish_project_kernel<<<(unsigned)((total + threads - 1) / threads), threads, 0, stream>>>(
        partial, chunks, n, m, P, accumulate ? 1 : 0);
    return cudaGetLastError();
}

cudaError_t launch_finish_aggregate(const float *partial, int chunks, int32_t n, int32_t m, float *pbar,
                                    cudaStream_t stream) {
    finish_aggregate_kernel<<<(m + 31) / 32, dim3(32, n > kMaxGroup ? 32 : kMaxGroup), 0, stream>>>(
        partial, chunks, n, m, pbar);
    return cudaGetLastError();
}

cudaError_t launch_aggregate(const float *P, int32_t n, int32_t m, float *pbar, cudaStream_t stream) {
    const int threads = 128;
    aggregate_kernel<<<(m + threads - 1) / threads, threads, 0, stream>>>(P, n, m, pbar);
    return cudaGetLastError();
}

}  // namespace core
