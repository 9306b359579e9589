// Device-side common random generator of the CORE library (sm_100a).
//
// The paper only requires that all machines share a generator of fresh
// N(0, I_d) vectors (Algorithm 1, first step).  Here that generator is
// Philox4x32-10 (Salmon et al., SC'11) followed by Box-Muller:
//   key     = (seed lo, seed hi)
//   counter = (q lo, q hi, j, t)   q = coordinate block k >> 2, j = vector, t = round
//   u(w)    = ((w >> 9) + 1/2) 2^-23
//   pair    = sqrt(-2 ln u(w_even)) * (cos, sin)(2 pi u(w_odd))
// One counter yields xi_j[4q .. 4q+3].  Nothing here touches memory: both the
// projection and the reconstruction kernel call these functions and so see
// identical vectors.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

namespace core {

constexpr uint32_t kPhiloxMulA = 0xD2511F53u;  // multiplies counter word 0
constexpr uint32_t kPhiloxMulB = 0xCD9E8D57u;  // multiplies counter word 2
constexpr uint32_t kPhiloxKeyA = 0x9E3779B9u;  // key word 0 increment per round
constexpr uint32_t kPhiloxKeyB = 0xBB67AE85u;  // key word 1 increment per round

// Key schedule, expanded once on the host: a[r], b[r] are the key words of round r.
struct RoundKeys {
    uint32_t a[10];
    uint32_t b[10];
};

inline RoundKeys expand_keys(uint64_t seed) {
    RoundKeys k;
    uint32_t a = (uint32_t)(seed & 0xFFFFFFFFu), b = (uint32_t)(seed >> 32);
    for (int r = 0; r < 10; ++r) {
        k.a[r] = a;
        k.b[r] = b;
        a += kPhiloxKeyA;
        b += kPhiloxKeyB;
    }
    return k;
}

__device__ __forceinline__ void mul_wide(uint32_t mult, uint32_t x, uint32_t &hi, uint32_t &lo) {
    unsigned long long p;
    asm("mul.wide.u32 %0, %1, %2;" : "=l"(p) : "r"(x), "r"(mult));
    lo = (uint32_t)p;
    hi = (uint32_t)(p >> 32);
}

// One Philox round.
__device__ __forceinline__ void philox_round(uint32_t &c0, uint32_t &c1, uint32_t &c2, uint32_t &c3,
                                             uint32_t ka, uint32_t kb) {
    uint32_t hi_a, lo_a, hi_b, lo_b;
    mul_wide(kPhiloxMulA, c0, hi_a, lo_a);
    mul_wide(kPhiloxMulB, c2, hi_b, lo_b);
    c0 = hi_b ^ c1 ^ ka;
    c1 = lo_b;
    c2 = hi_a ^ c3 ^ kb;
    c3 = lo_a;
}

// Rounds FIRST..9 on a counter that has already been through rounds 0..FIRST-1.
template <int FIRST>
__device__ __forceinline__ void philox_finish(uint32_t &c0, uint32_t &c1, uint32_t &c2, uint32_t &c3,
                                              const RoundKeys &k) {
#pragma unroll
    for (int r = FIRST; r < 10; ++r) philox_round(c0, c1, c2, c3, k.a[r], k.b[r]);
}

// Plain ten-round evaluation (used where speed does not matter).
__device__ __forceinline__ uint4 philox4x32_10(uint32_t q_lo, uint32_t q_hi, uint32_t j, uint32_t t,
                                               const RoundKeys &k) {
    uint32_t c0 = q_lo, c1 = q_hi, c2 = j, c3 = t;
    philox_finish<0>(c0, c1, c2, c3, k);
    return make_uint4(c0, c1, c2, c3);
}

// ---- split evaluation of the first two rounds ------------------------------------
// After round 0 the counter is (hiB(j)^q_hi^a0, loB(j), hiA(q_lo)^t^b0, loA(q_lo)):
// words 0,1 depend only on (j, q_hi), words 2,3 only on (q_lo, t).  Round 1 then
// needs MulA * word0 (a function of j, q_hi) and MulB * word2 (a function of q_lo, t).
// A kernel that keeps j fixed while q varies, or q fixed while j varies, evaluates
// the invariant half once.

struct JPart {       // depends on (j, q_hi)
    uint32_t x0;     // loB(j) ^ a1: xored with hiB(word 2) gives word 0 after round 1
    uint32_t x2;     // hiA(word 0 after round 0) ^ b1: xored with word 3 gives word 2 after round 1
    uint32_t w3;     // loA(word 0 after round 0) = word 3 after round 1
};

struct QPart {       // depends on (q_lo, t)
    uint32_t hi_b;   // hiB(word 2 after round 0)
    uint32_t lo_b;   // loB(word 2 after round 0) = word 1 after round 1
    uint32_t w3;     // loA(q_lo) = word 3 after round 0
};

__device__ __forceinline__ JPart philox_jpart(uint32_t j, uint32_t q_hi, const RoundKeys &k) {
    uint32_t hi_b, lo_b, hi_a, lo_a;
    mul_wide(kPhiloxMulB, j, hi_b, lo_b);
    uint32_t w0 = hi_b ^ q_hi ^ k.a[0];
    mul_wide(kPhiloxMulA, w0, hi_a, lo_a);
    JPart p;
    p.x0 = lo_b ^ k.a[1];
    p.x2 = hi_a ^ k.b[1];
    p.w3 = lo_a;
    return p;
}

__device__ __forceinline__ QPart philox_qpart(uint32_t q_lo, uint32_t t, const RoundKeys &k) {
    uint32_t hi_a, lo_a;
    mul_wide(kPhiloxMulA, q_lo, hi_a, lo_a);
    uint32_t w2 = hi_a ^ t ^ k.b[0];
    QPart p;
    mul_wide(kPhiloxMulB, w2, p.hi_b, p.lo_b);
    p.w3 = lo_a;
    return p;
}

__device__ __forceinline__ uint4 philox_combine(const JPart &jp, const QPart &qp, const RoundKeys &k) {
    uint32_t c0 = qp.hi_b ^ jp.x0;
    uint32_t c1 = qp.lo_b;
    uint32_t c2 = jp.x2 ^ qp.w3;
    uint32_t c3 = jp.w3;
    philox_finish<2>(c0, c1, c2, c3, k);
    return make_uint4(c0, c1, c2, c3);
}

// ---- Box-Muller ---------------------------------------------------------------------

// r = sqrt(-2 ln u), u = ((w >> 9) + 1/2) 2^-23, absolute error below 1e-6.
// u is formed exactly.  Away from 1 the hardware log2 is accurate enough; close to
// 1 its absolute error would dominate ln u, so -2 ln(1 - v), v = 1 - u (exact), is
// summed from its series instead.
__device__ __forceinline__ float bm_radius(uint32_t w) {
    float one_plus = __uint_as_float((w >> 9) | 0x3F800000u);   // 1 + k 2^-23
    float u = one_plus - 0.99999994f;                           // exact: (k + 1/2) 2^-23
    float lg;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(lg) : "f"(u));
    float l_far = lg * -1.3862943611198906f;                    // -2 ln 2 * log2 u
    float v = 1.0f - u;                                         // exact
    // -2 ln(1-v) = 2v + v^2 + (2/3) v^3 + (1/2) v^4 + ...
    float s = fmaf(v, 0.5f, 0.6666667f);
    s = fmaf(s, v, 1.0f);
    s = fmaf(s, v, 2.0f);
    float l_near = s * v;
    float l = (v < 0.03125f) ? l_near : l_far;
    float r;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(l));
    return r;
}

// (cos, sin)(2 pi u) scaled by r.  The angle is reduced exactly, in integers, to a
// quarter turn index and y in (-1, 1) with theta = quadrant * pi/2 + y * pi/4; sine and
// cosine of y pi/4 come from odd/even minimax polynomials in y (absolute error < 1e-7).
__device__ __forceinline__ float2 bm_pair(uint32_t w_radius, uint32_t w_angle) {
    float r = bm_radius(w_radius);
    uint32_t rot = w_angle + 0x20000000u;                       // + 1/8 turn, wraps with the circle
    // bits 29..9 of rot, doubled plus one, as the mantissa of a float in [4, 6):
    // 4 + (f + 1/2) 2^-20 with f the 21-bit fraction of the quarter turn.
    float y = __uint_as_float(((rot >> 8) & 0x003FFFFEu) | 0x40800001u) - 5.0f;   // exact
    float y2 = y * y;
    float sp = fmaf(-3.587725950637832e-05f, y2, 0.002489872043952346f);
    sp = fmaf(sp, y2, -0.08074536919593811f);
    sp = fmaf(sp, y2, 0.7853981256484985f);
    float sn = sp * y;
    float cp = fmaf(3.5313344142196e-06f, y2, -0.00032594200456514955f);
    cp = fmaf(cp, y2, 0.015854327008128166f);
    cp = fmaf(cp, y2, -0.3084251284599304f);
    float cs = fmaf(cp, y2, 1.0f);
    // quadrant: bit 30 of rot turns (cos, sin) into (-sin, cos); bit 31 negates both.
    bool odd = (rot & 0x40000000u) != 0u;
    float c = odd ? -sn : cs;
    float s = odd ? cs : sn;
    float rs = __uint_as_float(__float_as_uint(r) ^ (rot & 0x80000000u));
    return make_float2(rs * c, rs * s);
}

__device__ __forceinline__ float4 box_muller4(uint4 w) {
    float2 a = bm_pair(w.x, w.y);
    float2 b = bm_pair(w.z, w.w);
    return make_float4(a.x, a.y, b.x, b.y);
}

}  // namespace core
