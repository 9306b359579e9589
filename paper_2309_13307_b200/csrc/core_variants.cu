// Small kernels of the optimiser variants built on the round: the step rule of Algorithm 3's Option I
// (chosen on the device from the size of the combined messages) and the gossip averaging of
// Algorithm 5 (decentralised CORE-GD).  Everything here works on n x m or m numbers: microseconds.
#include "core_internal.h"

namespace core {

namespace {

constexpr int kVarThreads = 256;

// p = sqrt((1/m) sum_j pbar_j^2) and h = min{ m / (16 r1), c H^-1/2 p^-1/2 d^-3/4 m^3/4 }.
// One CTA; thread t sums entries t, t + 256, ... in ascending order, the 256 partial sums are added in
// ascending order by thread 0: a fixed order, in double (m numbers, nothing to save in fp32).
__global__ void option1_step_kernel(const float *__restrict__ pbar, int m, double d, double r1, double H, double c,
                                    float *p_out, float *h_out) {
    __shared__ double part[kVarThreads];
    double s = 0.0;
    for (int j = threadIdx.x; j < m; j += kVarThreads) s += (double)pbar[j] * (double)pbar[j];
    part[threadIdx.x] = s;
    __syncthreads();
    if (threadIdx.x != 0) return;
    double total = 0.0;
    for (int r = 0; r < kVarThreads; ++r) total += part[r];
    const double p = sqrt(total / (double)m);
    const double first = (double)m / (16.0 * r1);
    // p = 0 (no gradient at all) makes the second term infinite: the first one decides
    const double second = c * rsqrt(H) * rsqrt(p) * pow(d, -0.75) * pow((double)m, 0.75);
    *h_out = (float)(first < second ? first : second);
    if (p_out) *p_out = (float)p;
}

// One gossip round: out[i][j] = sum_l W[i][l] in[l][j], l ascending.
__global__ void gossip_round_kernel(const float *__restrict__ W, const float *__restrict__ in, int n, int m,
                                    float *__restrict__ out) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int i = blockIdx.y;
    if (j >= m) return;
    float s = 0.f;
    for (int l = 0; l < n; ++l) s = fmaf(W[(int64_t)i * n + l], in[(int64_t)l * m + j], s);
    out[(int64_t)i * m + j] = s;
}

// spread[0] = max over machines i and vectors j of |P[i][j] - P[reader][j]| (a maximum: order-free).
__global__ void consensus_spread_kernel(const float *__restrict__ P, int n, int m, int reader, float *spread) {
    __shared__ float part[kVarThreads];
    float worst = 0.f;
    for (int64_t e = threadIdx.x; e < (int64_t)n * m; e += kVarThreads)
        worst = fmaxf(worst, fabsf(P[e] - P[(int64_t)reader * m + e % m]));
    part[threadIdx.x] = worst;
    __syncthreads();
    if (threadIdx.x != 0) return;
    for (int r = 1; r < kVarThreads; ++r) worst = fmaxf(worst, part[r]);
    *spread = worst;
}

}  // namespace

cudaError_t launch_option1_step(const float *pbar, int32_t m, int64_t d, double r1, double H, double c, float *p_out,
                                float *h_out, cudaStream_t stream) {
    option1_step_kernel<<<1, kVarThreads, 0, stream>>>(pbar, m, (double)d, r1, H, c, p_out, h_out);
    return cudaGetLastError();
}

cudaError_t launch_gossip_round(const float *W, const float *in, int32_t n, int32_t m, float *out, cudaStream_t stream) {
    dim3 grid((unsigned)((m + 127) / 128), (unsigned)n);
    gossip_round_kernel<<<grid, 128, 0, stream>>>(W, in, n, m, out);
    return cudaGetLastError();
}

cudaError_t launch_consensus_spread(const float *P, int32_t n, int32_t m, int32_t reader, float *spread,
                                    cudaStream_t stream) {
    consensus_spread_kernel<<<1, kVarThreads, 0, stream>>>(P, n, m, reader, spread);
    return cudaGetLastError();
}

}  // namespace core
