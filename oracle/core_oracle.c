/*
 * CORE oracle -- TEST INFRASTRUCTURE, not a product path (see core_oracle.h).
 *
 * Everything is written out the long way, in fp64, one coordinate and one
 * vector at a time, in the order the paper states the operations:
 * Algorithm 1 (project, reconstruct), Algorithm 2 (CORE-GD), and the n-machine
 * estimator of Section 4.  No blocking, no fusion, no threads.
 */
#include "core_oracle.h"

#include <math.h>
#include <stddef.h>
#include <string.h>

/* ---- Philox4x32-10 (Salmon et al., SC'11) -------------------------------- */

#define PHILOX_MUL_A 0xD2511F53u /* multiplier applied to counter word 0 */
#define PHILOX_MUL_B 0xCD9E8D57u /* multiplier applied to counter word 2 */
#define PHILOX_KEY_A 0x9E3779B9u /* key word 0 increment (golden ratio) */
#define PHILOX_KEY_B 0xBB67AE85u /* key word 1 increment (sqrt 3 - 1)   */

void oracle_philox_round(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint64_t prod_a = (uint64_t)PHILOX_MUL_A * (uint64_t)ctr[0];
    uint64_t prod_b = (uint64_t)PHILOX_MUL_B * (uint64_t)ctr[2];
    uint32_t hi_a = (uint32_t)(prod_a >> 32), lo_a = (uint32_t)prod_a;
    uint32_t hi_b = (uint32_t)(prod_b >> 32), lo_b = (uint32_t)prod_b;
    uint32_t r0 = hi_b ^ ctr[1] ^ key[0];
    uint32_t r1 = lo_b;
    uint32_t r2 = hi_a ^ ctr[3] ^ key[1];
    uint32_t r3 = lo_a;
    out[0] = r0;
    out[1] = r1;
    out[2] = r2;
    out[3] = r3;
}

void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c[4] = {ctr[0], ctr[1], ctr[2], ctr[3]};
    uint32_t k[2] = {key[0], key[1]};
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { /* the key is bumped before every round but the first */
            k[0] += PHILOX_KEY_A;
            k[1] += PHILOX_KEY_B;
        }
        uint32_t next[4];
        oracle_philox_round(c, k, next);
        memcpy(c, next, sizeof c);
    }
    memcpy(out, c, sizeof c);
}

/* ---- common Gaussian vectors ---------------------------------------------- */

double oracle_uniform(uint32_t w) {
    return ((double)(w >> 9) + 0.5) * (1.0 / 8388608.0); /* 2^-23 */
}

void oracle_xi_words(uint64_t seed, uint32_t t, uint32_t j, uint64_t q, uint32_t w[4]) {
    uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
    uint32_t ctr[4] = {(uint32_t)(q & 0xFFFFFFFFu), (uint32_t)(q >> 32), j, t};
    oracle_philox4x32_10(ctr, key, w);
}

void oracle_box_muller(const uint32_t w[4], double z[4]) {
    const double two_pi = 6.283185307179586476925286766559;
    for (int pair = 0; pair < 2; ++pair) {
        double u_radius = oracle_uniform(w[2 * pair]);
        double u_angle = oracle_uniform(w[2 * pair + 1]);
        double r = sqrt(-2.0 * log(u_radius));
        double theta = two_pi * u_angle;
        z[2 * pair] = r * cos(theta);
        z[2 * pair + 1] = r * sin(theta);
    }
}

void oracle_xi_block(uint64_t seed, uint32_t t, uint32_t j, uint64_t q, double z[4]) {
    uint32_t w[4];
    oracle_xi_words(seed, t, j, q, w);
    oracle_box_muller(w, z);
}

static double xi_at(uint64_t seed, uint32_t t, uint32_t j, int64_t k) {
    double z[4];
    oracle_xi_block(seed, t, j, (uint64_t)k >> 2, z);
    return z[k & 3];
}

void oracle_xi_range(uint64_t seed, uint32_t t, uint32_t j, int64_t k0, int64_t k1, double *out) {
    for (int64_t k = k0; k < k1; ++k) out[k - k0] = xi_at(seed, t, j, k);
}

/* convenience loops over the two functions above, for checking many blocks at once */
void oracle_xi_words_many(uint64_t seed, uint32_t t, uint32_t j, uint64_t q0, int64_t nq, uint32_t *out) {
    for (int64_t r = 0; r < nq; ++r) oracle_xi_words(seed, t, j, q0 + (uint64_t)r, out + 4 * r);
}

void oracle_box_muller_many(const uint32_t *w, int64_t nb, double *z) {
    for (int64_t r = 0; r < nb; ++r) oracle_box_muller(w + 4 * r, z + 4 * r);
}

/* ---- gradient element access ---------------------------------------------- */

/* dtype 0 float, 1 bfloat16 bit pattern (upper half of an fp32), 2 double. */
static double grad_at(const void *g, int dtype, int64_t k) {
    if (dtype == 0) return (double)((const float *)g)[k];
    if (dtype == 1) {
        uint32_t bits = (uint32_t)((const uint16_t *)g)[k] << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    return ((const double *)g)[k];
}

static size_t grad_elem_size(int dtype) { return dtype == 0 ? 4 : (dtype == 1 ? 2 : 8); }

/* ---- Algorithm 1: project -------------------------------------------------- */

double oracle_project_slice(uint64_t seed, uint32_t t, uint32_t j, const void *g, int dtype,
                            int64_t k0, int64_t k1) {
    double p = 0.0;
    int64_t k = k0;
    while (k < k1) {
        /* one generator call serves the (up to four) coordinates of a block */
        double z[4];
        oracle_xi_block(seed, t, j, (uint64_t)k >> 2, z);
        int64_t block_end = (k | 3) + 1;
        if (block_end > k1) block_end = k1;
        for (; k < block_end; ++k) p += grad_at(g, dtype, k) * z[k & 3];
    }
    return p;
}

void oracle_project(uint64_t seed, uint32_t t, int64_t d, int32_t m, int32_t n, const void *G,
                    int dtype, int64_t ldg, double *P) {
    for (int32_t i = 0; i < n; ++i) {
        const char *row = (const char *)G + (size_t)i * (size_t)ldg * grad_elem_size(dtype);
        for (int32_t j = 0; j < m; ++j)
            P[(size_t)i * m + j] = oracle_project_slice(seed, t, (uint32_t)j, row, dtype, 0, d);
    }
}

/* ---- Algorithm 2, third step: the central machine combines the messages ---- */

void oracle_aggregate(const double *P, int32_t n, int32_t m, double *pbar) {
    for (int32_t j = 0; j < m; ++j) {
        double s = 0.0;
        for (int32_t i = 0; i < n; ++i) s += P[(size_t)i * m + j];
        pbar[j] = s / (double)n;
    }
}

/* ---- Algorithm 1: reconstruct ---------------------------------------------- */

void oracle_reconstruct_slice(uint64_t seed, uint32_t t, int32_t m, const double *pbar, int64_t k0,
                              int64_t k1, double *out) {
    /* block by block (one generator call yields four coordinates); within a
     * block every coordinate's sum runs over j = 0..m-1 in order */
    for (int64_t q = k0 >> 2; q * 4 < k1; ++q) {
        double s[4] = {0.0, 0.0, 0.0, 0.0};
        for (int32_t j = 0; j < m; ++j) {
            double z[4];
            oracle_xi_block(seed, t, (uint32_t)j, (uint64_t)q, z);
            for (int l = 0; l < 4; ++l) s[l] += pbar[j] * z[l];
        }
        for (int l = 0; l < 4; ++l) {
            int64_t k = q * 4 + l;
            if (k >= k0 && k < k1) out[k - k0] = s[l] / (double)m;
        }
    }
}

/* ---- least-squares objective and Algorithm 2 ------------------------------- */

double oracle_ls_loss(const float *A, const float *b, int32_t n, int32_t rows, int64_t d,
                      const double *x) {
    double f = 0.0;
    for (int32_t i = 0; i < n; ++i) {
        double sq = 0.0;
        for (int32_t r = 0; r < rows; ++r) {
            const float *a = A + ((size_t)i * rows + r) * (size_t)d;
            double res = -(double)b[(size_t)i * rows + r];
            for (int64_t k = 0; k < d; ++k) res += (double)a[k] * x[k];
            sq += res * res;
        }
        f += sq / (2.0 * (double)rows);
    }
    return f / (double)n;
}

void oracle_ls_grad(const float *A, const float *b, int32_t n, int32_t rows, int64_t d,
                    const double *x, double *G) {
    for (int32_t i = 0; i < n; ++i) {
        double *g = G + (size_t)i * (size_t)d;
        for (int64_t k = 0; k < d; ++k) g[k] = 0.0;
        for (int32_t r = 0; r < rows; ++r) {
            const float *a = A + ((size_t)i * rows + r) * (size_t)d;
            double res = -(double)b[(size_t)i * rows + r];
            for (int64_t k = 0; k < d; ++k) res += (double)a[k] * x[k];
            for (int64_t k = 0; k < d; ++k) g[k] += (double)a[k] * res;
        }
        for (int64_t k = 0; k < d; ++k) g[k] /= (double)rows;
    }
}

void oracle_gd_step(uint64_t seed, uint32_t t, int32_t m, const float *A, const float *b, int32_t n,
                    int32_t rows, int64_t d, double h, double *x, double *work, int exact) {
    double *G = work;                      /* n*d */
    double *P = G + (size_t)n * (size_t)d; /* n*m */
    double *pbar = P + (size_t)n * m;      /* m   */
    double *gt = pbar + m;                 /* d   */

    oracle_ls_grad(A, b, n, rows, d, x, G);
    if (exact) {
        /* gradient of f = (1/n) sum_i f_i, no compression */
        for (int64_t k = 0; k < d; ++k) {
            double s = 0.0;
            for (int32_t i = 0; i < n; ++i) s += G[(size_t)i * d + k];
            gt[k] = s / (double)n;
        }
    } else {
        oracle_project(seed, t, d, m, n, G, 2, d, P);
        oracle_aggregate(P, n, m, pbar);
        oracle_reconstruct_slice(seed, t, m, pbar, 0, d, gt);
    }
    for (int64_t k = 0; k < d; ++k) x[k] -= h * gt[k];
}

/* ---- Algorithm 4: CORE-AGD (heavy ball with the CORE gradient estimate) ------ */

void oracle_agd_step(uint64_t seed, uint32_t t, int32_t m, const float *A, const float *b, int32_t n,
                     int32_t rows, int64_t d, double h, double beta, double *x, double *x_prev,
                     double *work, int exact) {
    double *y = work; /* d doubles, then the gd-step work area */
    double *rest = work + d;
    /* look-ahead point y^k = x^k + (1 - beta)(x^k - x^{k-1}) */
    for (int64_t k = 0; k < d; ++k) y[k] = x[k] + (1.0 - beta) * (x[k] - x_prev[k]);
    /* x^{k+1} = y^k - h * gradient estimate at y^k: a CORE-GD step taken from y */
    oracle_gd_step(seed, t, m, A, b, n, rows, d, h, y, rest, exact);
    for (int64_t k = 0; k < d; ++k) {
        x_prev[k] = x[k];
        x[k] = y[k];
    }
}

/* ---- Algorithm 3: CORE-GD with the comparison step ---------------------------- */

int oracle_gd_step_guarded(uint64_t seed, uint32_t t, int32_t m, const float *A, const float *b, int32_t n,
                           int32_t rows, int64_t d, double h, double *x, double *f_x, double *work) {
    double *trial = work; /* d doubles, then the gd-step work area */
    double *rest = work + d;
    for (int64_t k = 0; k < d; ++k) trial[k] = x[k];
    /* trial point x~ = x - h * gradient estimate at x */
    oracle_gd_step(seed, t, m, A, b, n, rows, d, h, trial, rest, 0);
    /* x^{k+1} = argmin over {x^k, x~} of f; a tie keeps x^k */
    double f_trial = oracle_ls_loss(A, b, n, rows, d, trial);
    if (f_trial < *f_x) {
        for (int64_t k = 0; k < d; ++k) x[k] = trial[k];
        *f_x = f_trial;
        return 1;
    }
    return 0;
}

/* ---- Algorithm 3, Option I: the step chosen from the size of the messages ------ */

double oracle_message_norm(const double *pbar, int32_t m) {
    double sum_sq = 0.0;
    for (int32_t j = 0; j < m; ++j) sum_sq += pbar[j] * pbar[j];
    return sqrt(sum_sq / (double)m);
}

double oracle_option1_step(double p, int32_t m, int64_t d, double r1, double H, double c) {
    double first = (double)m / (16.0 * r1);
    /* c * H^(-1/2) * p^(-1/2) * d^(-3/4) * m^(3/4); p = 0 (no gradient) makes it infinite */
    double second = c * pow(H, -0.5) * pow(p, -0.5) * pow((double)d, -0.75) * pow((double)m, 0.75);
    return first < second ? first : second;
}

int oracle_gd_step_option1(uint64_t seed, uint32_t t, int32_t m, const float *A, const float *b, int32_t n,
                           int32_t rows, int64_t d, double r1, double H, double c, double *x, double *f_x,
                           double *p_out, double *h_out, double *work) {
    double *G = work;                      /* n*d */
    double *P = G + (size_t)n * (size_t)d; /* n*m */
    double *pbar = P + (size_t)n * m;      /* m   */
    double *gt = pbar + m;                 /* d   */
    double *trial = gt + d;                /* d   */

    /* the round: machine i sends p_ij, the central machine combines, everyone reconstructs */
    oracle_ls_grad(A, b, n, rows, d, x, G);
    oracle_project(seed, t, d, m, n, G, 2, d, P);
    oracle_aggregate(P, n, m, pbar);
    oracle_reconstruct_slice(seed, t, m, pbar, 0, d, gt);
    /* the statistic p of the combined messages and the step it selects */
    double p = oracle_message_norm(pbar, m);
    double h = oracle_option1_step(p, m, d, r1, H, c);
    if (p_out) *p_out = p;
    if (h_out) *h_out = h;
    /* trial point and comparison step; a tie keeps x */
    for (int64_t k = 0; k < d; ++k) trial[k] = x[k] - h * gt[k];
    double f_trial = oracle_ls_loss(A, b, n, rows, d, trial);
    if (f_trial < *f_x) {
        for (int64_t k = 0; k < d; ++k) x[k] = trial[k];
        *f_x = f_trial;
        return 1;
    }
    return 0;
}

/* ---- Algorithm 5: decentralised CORE-GD ----------------------------------------- */

void oracle_gossip_round(const double *W, const double *P, int32_t n, int32_t m, double *P_next) {
    for (int32_t i = 0; i < n; ++i)
        for (int32_t j = 0; j < m; ++j) {
            double s = 0.0;
            for (int32_t l = 0; l < n; ++l) s += W[(size_t)i * n + l] * P[(size_t)l * m + j];
            P_next[(size_t)i * m + j] = s;
        }
}

void oracle_gossip_average(const double *W, int32_t rounds, int32_t n, int32_t m, double *P, double *scratch) {
    for (int32_t r = 0; r < rounds; ++r) {
        oracle_gossip_round(W, P, n, m, scratch);
        memcpy(P, scratch, (size_t)n * m * sizeof(double));
    }
}

double oracle_decentralized_step(uint64_t seed, uint32_t t, int32_t m, const float *A, const float *b, int32_t n,
                                 int32_t rows, int64_t d, const double *W, int32_t rounds, int32_t reader,
                                 int as_printed, double h, double *x, double *work) {
    double *G = work;                      /* n*d */
    double *P = G + (size_t)n * (size_t)d; /* n*m */
    double *scratch = P + (size_t)n * m;   /* n*m */
    double *gt = scratch + (size_t)n * m;  /* d   */

    /* machine i computes its projections locally */
    oracle_ls_grad(A, b, n, rows, d, x, G);
    oracle_project(seed, t, d, m, n, G, 2, d, P);
    /* the m-dimensional averaging problem, solved approximately by gossip: row i becomes machine i's
     * estimate of p = (1/n) sum_i p_i */
    oracle_gossip_average(W, rounds, n, m, P, scratch);
    const double *p = P + (size_t)reader * m;
    double spread = 0.0;
    for (int32_t i = 0; i < n; ++i)
        for (int32_t j = 0; j < m; ++j) {
            double dev = fabs(P[(size_t)i * m + j] - p[j]);
            if (dev > spread) spread = dev;
        }
    /* reconstruction from the consensus value, prefactor 1/m (mean reading) or n/m (as printed) */
    oracle_reconstruct_slice(seed, t, m, p, 0, d, gt);
    double prefactor = as_printed ? (double)n : 1.0;
    for (int64_t k = 0; k < d; ++k) x[k] -= h * prefactor * gt[k];
    return spread;
}
