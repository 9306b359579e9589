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
// the invariant half once.  The 32x32->64 multiply is the scarcest resource of the
// generator on this GPU (a quarter of the fp32 rate), so this saves real time.

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
// One call turns the four words of a counter into four Gaussians.  The two pairs are
// evaluated side by side in packed fp32 (fma.rn.f32x2 and friends), which halves the
// instruction count of the floating-point part.  On this GPU the fp32 pipe also executes
// the wide multiplies of Philox, so the split of the work between pipes matters: bit
// manipulation (integer pipe) is preferred over floating-point arithmetic where both can
// do the job.
//
// Radius.  u = (k + 1/2) 2^-23 is formed exactly by inserting k = w >> 9 under the
// exponent of 1.0 (one funnel shift) and subtracting 1 - 2^-24.  S = sqrt(-log2 u) comes
// from the hardware log2 and square root; r = sqrt(2 ln 2) S, and that constant is folded
// into the sine/cosine polynomials.  The hardware log2 has an absolute error of about
// 2e-7, harmless except when u is close to 1 (log u close to 0): for v = 1 - u < 2^-10
// (v is exact) the series of -log2(1 - v) replaces it.  That case is rare (one radius in
// 1024), so it sits behind a branch tested once per call.
//
// Angle.  theta = 2 pi u = pi (h + f) with h = bit 31 of the word (which half turn) and
// f = (bits 30..9 + 1/2) / 2^22 in (0, 1).  Those 22 bits, doubled plus one, inserted under
// the exponent of 1.0, minus 1.5, are y = f - 1/2 in (-1/2, 1/2) exactly, and
//   cos theta = -(-1)^h sin(pi y),   sin theta = (-1)^h cos(pi y):
// odd/even minimax polynomials in y (the minus sits in the odd one's coefficients), and bit
// 31 is xored into the sign of S.  No integer arithmetic on the word beyond the bit insert.
//
// Worst absolute error over all 2^23 radius words and all 2^23 angle words: 1.2e-6.

constexpr uint32_t kNearOneWord = 0xFFC00000u;   // words with v = 1 - u < 2^-10

// -log2(1 - v) = (v + v^2/2 + v^3/3 + v^4/4 + ...) / ln 2
__device__ __forceinline__ float bm_near_one(float v) {
    float s = fmaf(v, 0.36067376f, 0.48089835f);
    s = fmaf(s, v, 0.72134752f);
    s = fmaf(s, v, 1.44269504f);
    return s * v;
}

__device__ __forceinline__ float2 bm_splat(float c) { return make_float2(c, c); }

// log2 u (negative) of the two radius words of a call (lanes x, y = pair a, pair b) by the
// hardware log2; u itself is returned for the rare correction.
__device__ __forceinline__ float2 bm_log2(uint4 w, float2 &u) {
    u = __fadd2_rn(make_float2(__uint_as_float(__funnelshift_r(w.x, 0x7Fu, 9)),
                               __uint_as_float(__funnelshift_r(w.z, 0x7Fu, 9))),
                   bm_splat(-0.99999994f));
    float2 l;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(l.x) : "f"(u.x));
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(l.y) : "f"(u.y));
    return l;
}

__device__ __forceinline__ void bm_fix_near_one(uint4 w, float2 u, float2 &l) {
    if (w.x >= kNearOneWord) l.x = bm_near_one(1.0f - u.x);
    if (w.z >= kNearOneWord) l.y = bm_near_one(1.0f - u.y);
}

// The rest of Box-Muller given l with |l| = -log2 u of the two pairs (the sign of l is ignored:
// the hardware path delivers log2 u < 0, the correction delivers the positive series), as its factors:
// with S = (-1)^h sqrt(-log2 u) the pair is (r cos theta, r sin theta) = ((S y) sp, S cs).  Lanes x, y of
// every member = pair a, pair b.  A consumer that multiplies the values by a number p of its own can let p
// meet S first, ((p S) y) sp and (p S) cs, and save the two products that would form the values; with
// p = 1 that is bit for bit what bm_finish returns.
struct BmParts {
    float2 s;     // (-1)^h sqrt(-log2 u)
    float2 y;     // f - 1/2
    float2 sp;    // -sqrt(2 ln 2) sin(pi y) / y
    float2 cs;    //  sqrt(2 ln 2) cos(pi y)
};

__device__ __forceinline__ BmParts bm_parts(uint4 w, float2 l) {
    BmParts r;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r.s.x) : "f"(fabsf(l.x)));
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r.s.y) : "f"(fabsf(l.y)));

    // angles: theta = pi (h + f), h = bit 31 of the word, f = (bits 30..9 + 1/2) / 2^22 in (0, 1).
    // With y = f - 1/2:  cos theta = -(-1)^h sin(pi y),  sin theta = (-1)^h cos(pi y).
    r.y = __fadd2_rn(make_float2(__uint_as_float(((w.y >> 8) & 0x007FFFFEu) | 0x3F800001u),
                                 __uint_as_float(((w.w >> 8) & 0x007FFFFEu) | 0x3F800001u)),
                     bm_splat(-1.5f));
    r.s.x = __uint_as_float(__float_as_uint(r.s.x) ^ (w.y & 0x80000000u));
    r.s.y = __uint_as_float(__float_as_uint(r.s.y) ^ (w.w & 0x80000000u));
    const float2 y2 = __fmul2_rn(r.y, r.y);
    // -sqrt(2 ln 2) sin(pi y) / y and sqrt(2 ln 2) cos(pi y)
    float2 sp = __ffma2_rn(bm_splat(-0.09091975539922714f), y2, bm_splat(0.7041443586349487f));
    sp = __ffma2_rn(sp, y2, bm_splat(-3.0024325847625732f));
    sp = __ffma2_rn(sp, y2, bm_splat(6.08450984954834f));
    r.sp = __ffma2_rn(sp, y2, bm_splat(-3.6989426612854004f));
    float2 cp = __ffma2_rn(bm_splat(0.2591251730918884f), y2, bm_splat(-1.568420648574829f));
    cp = __ffma2_rn(cp, y2, bm_splat(4.778461456298828f));
    cp = __ffma2_rn(cp, y2, bm_splat(-5.810277938842773f));
    r.cs = __ffma2_rn(cp, y2, bm_splat(1.1774100065231323f));
    return r;
}

__device__ __forceinline__ float4 bm_finish(uint4 w, float2 l) {
    const BmParts r = bm_parts(w, l);
    const float2 zs = __fmul2_rn(r.s, r.cs);                       // r sin theta
    const float2 zc = __fmul2_rn(__fmul2_rn(r.s, r.y), r.sp);      // r cos theta
    return make_float4(zc.x, zs.x, zc.y, zs.y);
}

// N calls at once: the rare near-one correction of all 2N radii sits behind one test, which
// leaves the N evaluations in one straight-line block for the instruction scheduler.
template <int N>
__device__ __forceinline__ void box_muller4xN(const uint4 (&w)[N], float4 (&z)[N]) {
    float2 u[N], l[N];
    uint32_t top = 0u;
#pragma unroll
    for (int c = 0; c < N; ++c) {
        l[c] = bm_log2(w[c], u[c]);
        top = __vimax3_u32(top, w[c].x, w[c].z);
    }
    if (top >= kNearOneWord) {
#pragma unroll
        for (int c = 0; c < N; ++c) bm_fix_near_one(w[c], u[c], l[c]);
    }
#pragma unroll
    for (int c = 0; c < N; ++c) z[c] = bm_finish(w[c], l[c]);
}

// The factors of N calls (same near-one handling as box_muller4xN).
template <int N>
__device__ __forceinline__ void box_muller_parts(const uint4 (&w)[N], BmParts (&r)[N]) {
    float2 u[N], l[N];
    uint32_t top = 0u;
#pragma unroll
    for (int c = 0; c < N; ++c) {
        l[c] = bm_log2(w[c], u[c]);
        top = __vimax3_u32(top, w[c].x, w[c].z);
    }
    if (top >= kNearOneWord) {
#pragma unroll
        for (int c = 0; c < N; ++c) bm_fix_near_one(w[c], u[c], l[c]);
    }
#pragma unroll
    for (int c = 0; c < N; ++c) r[c] = bm_parts(w[c], l[c]);
}

__device__ __forceinline__ float4 box_muller4(uint4 w) {
    const uint4 ws[1] = {w};
    float4 zs[1];
    box_muller4xN<1>(ws, zs);
    return zs[0];
}

}  // namespace core
