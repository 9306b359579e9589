/*
 * CORE oracle -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, single-threaded fp64 restatement of the CORE round
 * (Common Random Reconstruction: Algorithm 1, Algorithm 2 and the n-machine
 * estimator of Section 4 of the paper).  It exists so that the CUDA library can
 * be checked against something written independently from the paper.  Only the
 * test-suite, the smoke check and the benchmark's CPU-baseline leg may call it.
 * It shares no source, header, table or helper with the CUDA library.
 *
 * Common random vectors.  The paper only asks for "a common random number
 * generator" that yields fresh i.i.d. N(0, I_d) vectors each round
 * (Algorithm 1, first step).  This library fixes that generator as follows.
 *
 *   words   : Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) with
 *             key     = (seed mod 2^32, seed >> 32)
 *             counter = (q mod 2^32, q >> 32, j, t)
 *             q = k >> 2 the block of four coordinates, j the 0-based vector
 *             index, t the round ("fresh" vectors: a new t per round).
 *   uniform : u(w) = ((w >> 9) + 1/2) * 2^-23, in (0,1), exact in fp32 and fp64.
 *   normal  : Box-Muller on word pairs (w0,w1) and (w2,w3):
 *             r = sqrt(-2 ln u(w_even)), theta = 2 pi u(w_odd),
 *             xi_j[4q+0..3] = (r_a cos th_a, r_a sin th_a, r_b cos th_b, r_b sin th_b).
 *
 * Parity pins (tests/, CPU only): Philox against an arbitrary-precision integer
 * restatement, hand-evaluated rounds and the generator's published
 * known-answer vectors; the round against hand-expanded sums at d=8, m=3,
 * unit-vector probes, <gbar, gtilde> = (1/m) sum pbar_j^2, linearity, and the
 * estimator's first and second moments (Lemma 3.1, proof of Lemma 3.2); the message-norm statistic by
 * the law of the messages, Option I's step by its closed form, gossip by the spectrum of W (limit = the
 * centralised mean, contraction at the second eigenvalue) and a hand-worked three-machine example.
 */
#ifndef CORE_ORACLE_H
#define CORE_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Philox4x32-10: ten rounds on a 4-word counter with a 2-word key. */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);

/* A single Philox round (no key schedule step), exposed for hand checks. */
void oracle_philox_round(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);

/* u(w) = ((w >> 9) + 1/2) 2^-23. */
double oracle_uniform(uint32_t w);

/* Box-Muller on the word pairs (w0,w1), (w2,w3): four standard normals. */
void oracle_box_muller(const uint32_t w[4], double z[4]);

/* The four raw words behind xi_j^{(t)}[4q .. 4q+3]. */
void oracle_xi_words(uint64_t seed, uint32_t t, uint32_t j, uint64_t q, uint32_t w[4]);

/* xi_j^{(t)}[4q .. 4q+3] in fp64. */
void oracle_xi_block(uint64_t seed, uint32_t t, uint32_t j, uint64_t q, double z[4]);

/* xi_j^{(t)}[k0 .. k1) written to out[0 .. k1-k0). */
void oracle_xi_range(uint64_t seed, uint32_t t, uint32_t j, int64_t k0, int64_t k1, double *out);

/* out[4r..4r+3] = words of block q0 + r, r < nq. */
void oracle_xi_words_many(uint64_t seed, uint32_t t, uint32_t j, uint64_t q0, int64_t nq, uint32_t *out);

/* z[4r..4r+3] = Box-Muller of w[4r..4r+3], r < nb. */
void oracle_box_muller_many(const uint32_t *w, int64_t nb, double *z);

/*
 * Projection (Algorithm 1, "M1 sends p_i = <a, xi_i>"; Algorithm 2, machine i
 * sends p_ij): sum over k in [k0,k1) of g[k] * xi_j[k], k ascending, fp64.
 * g points at coordinate 0 of one machine's gradient.
 * dtype 0: g is float[]; dtype 1: g is bfloat16 bit patterns (uint16_t[]),
 * widened exactly.
 */
double oracle_project_slice(uint64_t seed, uint32_t t, uint32_t j, const void *g, int dtype,
                            int64_t k0, int64_t k1);

/* P[i*m + j] = <g_i, xi_j>, i < n, j < m; row i of G starts at element i*ldg. */
void oracle_project(uint64_t seed, uint32_t t, int64_t d, int32_t m, int32_t n, const void *G,
                    int dtype, int64_t ldg, double *P);

/*
 * Aggregation at the central machine (Algorithm 2, third step) in the mean
 * convention of the Section-4 estimator (prefactor 1/(nm)):
 * pbar[j] = (1/n) sum_i P[i*m + j], i ascending.
 */
void oracle_aggregate(const double *P, int32_t n, int32_t m, double *pbar);

/*
 * Reconstruction (Algorithm 1 last step; Eq. "reconstruction"):
 * out[k-k0] = (1/m) sum_j pbar[j] xi_j[k], k in [k0,k1), j ascending.
 */
void oracle_reconstruct_slice(uint64_t seed, uint32_t t, int32_t m, const double *pbar, int64_t k0,
                              int64_t k1, double *out);

/*
 * Least-squares objective of the CORE-GD driver:
 * f(x) = (1/n) sum_i 1/(2 rows) ||A_i x - b_i||^2, A is n x rows x d row-major
 * (ridge-separable form of Section 4 with a quadratic loss and no ridge term).
 */
double oracle_ls_loss(const float *A, const float *b, int32_t n, int32_t rows, int64_t d,
                      const double *x);

/* G[i*d + k] = (A_i^T (A_i x - b_i))[k] / rows. */
void oracle_ls_grad(const float *A, const float *b, int32_t n, int32_t rows, int64_t d,
                    const double *x, double *G);

/*
 * One CORE-GD iteration (Algorithm 2) on the least-squares objective with round
 * index t: x <- x - h * gtilde, gtilde the reconstruction of the mean of the
 * projected machine gradients.  work must hold n*d + n*m + m + d doubles.
 * exact != 0 bypasses the compression (plain gradient descent), for pins.
 */
void oracle_gd_step(uint64_t seed, uint32_t t, int32_t m, const float *A, const float *b, int32_t n,
                    int32_t rows, int64_t d, double h, double *x, double *work, int exact);

/*
 * One CORE-AGD iteration (Algorithm 4: heavy ball on top of the CORE estimate) with round
 * index t: y = x + (1 - beta)(x - x_prev); x_new = y - h * gtilde(y); then x_prev <- x,
 * x <- x_new.  The gradient is taken at y (the algorithm's title and update line say y; its
 * displayed reconstruction formula prints x, a typo).  work: d doubles more than gd_step needs.
 */
void oracle_agd_step(uint64_t seed, uint32_t t, int32_t m, const float *A, const float *b, int32_t n,
                     int32_t rows, int64_t d, double h, double beta, double *x, double *x_prev,
                     double *work, int exact);

/*
 * One iteration of the non-convex variant (Algorithm 3, "CORE-GD in Non-convex Optimization")
 * with a step h fixed by the caller (its Option II: h depends only on constants of the problem):
 * trial x~ = x - h * gtilde(x) with round index t, then x <- argmin over {x, x~} of f, a tie
 * keeping x.  *f_x holds f(x) on entry and f of the kept point on return.  Returns 1 if the
 * trial point was accepted.  Option I's step rule is not restated: the statistic it needs is
 * garbled in the algorithm's text.  work: d doubles more than gd_step needs.
 */
int oracle_gd_step_guarded(uint64_t seed, uint32_t t, int32_t m, const float *A, const float *b, int32_t n,
                           int32_t rows, int64_t d, double h, double *x, double *f_x, double *work);

/*
 * Algorithm 3 with Option I: the step is chosen from a statistic p of the combined messages.  The
 * algorithm prints p = (1/m) sum_{i<=m} (sum_{j<=n} p_ij): its index ranges are swapped, and a plain mean
 * of zero-mean Gaussians cannot bound the gradient norm as the proof of the theorem needs.  Reading
 * taken: the root mean square of the combined messages,
 *     p = sqrt((1/m) sum_j pbar_j^2),   pbar_j = (1/n) sum_i p_ij,
 * whose square has expectation ||mean gradient||^2 (the messages of a vector a are N(0, ||a||^2 I_m),
 * lemma on the law of the messages in the privacy appendix).
 */
double oracle_message_norm(const double *pbar, int32_t m);

/*
 * Option I's step: h = min{ m / (16 r1), c H^(-1/2) p^(-1/2) d^(-3/4) m^(3/4) } with r1 the bound on the
 * trace of the Hessian, H the Lipschitz constant of the Hessian and c the printed constant (1/1600).
 */
double oracle_option1_step(double p, int32_t m, int64_t d, double r1, double H, double c);

/*
 * One iteration of Algorithm 3 with Option I on the least-squares objective, in the algorithm's order:
 * round t (project, combine, reconstruct), p, h, trial point x - h * gtilde, comparison step (a tie keeps
 * x).  *f_x: f(x) on entry, f of the kept point on return; *p_out, *h_out (may be NULL) receive the
 * statistic and the step.  Returns 1 if the trial point was taken.  work: n*d + n*m + m + 2*d doubles.
 */
int oracle_gd_step_option1(uint64_t seed, uint32_t t, int32_t m, const float *A, const float *b, int32_t n,
                           int32_t rows, int64_t d, double r1, double H, double c, double *x, double *f_x,
                           double *p_out, double *h_out, double *work);

/*
 * Decentralised CORE-GD (appendix "Decentralized CORE Based Algorithms", Algorithm 5).  The machines
 * hold their messages p_i (rows of P, n x m) and obtain p = (1/n) sum_i p_i, the minimiser of the
 * m-dimensional problem (1/n) sum_i 1/2 ||x - p_i||^2, by exchanging with neighbours only.  Here that
 * solver is plain gossip averaging with a gossip matrix W (n x n, row-major, symmetric, doubly
 * stochastic, zero between machines that are not neighbours):
 *     one round:  P_next[i] = sum_l W[i][l] P[l]   (l ascending).
 * oracle_gossip_average runs `rounds` of them in place (scratch: n*m doubles).
 */
void oracle_gossip_round(const double *W, const double *P, int32_t n, int32_t m, double *P_next);
void oracle_gossip_average(const double *W, int32_t rounds, int32_t n, int32_t m, double *P, double *scratch);

/*
 * One iteration of Algorithm 5 on the least-squares objective with round index t: local projections,
 * `rounds` gossip rounds, reconstruction from machine `reader`'s estimate of p, x <- x - h * estimate.
 * as_printed = 0 reconstructs with prefactor 1/m (the mean convention of the Section-4 estimator, as
 * everywhere in this oracle); as_printed != 0 uses the printed n/m.  Returns the largest absolute
 * difference between any machine's estimate and the reader's (how far from consensus the gossip
 * stopped).  work: n*d + 2*n*m + d doubles.
 */
double oracle_decentralized_step(uint64_t seed, uint32_t t, int32_t m, const float *A, const float *b, int32_t n,
                                 int32_t rows, int64_t d, const double *W, int32_t rounds, int32_t reader,
                                 int as_printed, double h, double *x, double *work);

#ifdef __cplusplus
}
#endif
#endif
