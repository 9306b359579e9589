"""Pins for the oracle's project / aggregate / reconstruct (CPU only).

What fixes the expected values: Algorithm 1 and the Section-4 estimator written
out as explicit sums over a table of xi values (brute force, tiny sizes);
identities that follow from them; and the moments the paper proves
(Lemma 3.1: unbiased; proof of Lemma 3.2: E[xi xi^T A xi xi^T] = tr(A) I + 2A,
which at A = I gives E||a~||^2 = ((d+m+1)/m) ||a||^2; the DP appendix lemma:
the message p = Xi a is N(0, ||a||^2 I_m)).
"""
import math

import numpy as np
import pytest
import torch
from scipy import stats

import core_inputs
import oracle


def xi_table(seed, t, m, d):
    """xi[j][k] as nested Python lists, from the generator alone."""
    return [[float(v) for v in oracle.xi_range(seed, t, j, 0, d)] for j in range(m)]


def test_brute_force_d8_m3_n2():
    seed, t, d, m, n = 1, 0, 8, 3, 2
    G = core_inputs.gradients(n, d, seed=0).numpy()
    xi = xi_table(seed, t, m, d)           # the 24 numbers everything below is expanded from
    assert len(xi) == 3 and len(xi[0]) == 8
    # Algorithm 1 / Algorithm 2: p_ij = <g_i, xi_j>
    P = [[sum(float(G[i][k]) * xi[j][k] for k in range(d)) for j in range(m)] for i in range(n)]
    # Section-4 estimator: gtilde = 1/(n m) sum_i sum_j p_ij xi_j
    gt = [sum(P[i][j] * xi[j][k] for i in range(n) for j in range(m)) / (n * m) for k in range(d)]
    pbar = [sum(P[i][j] for i in range(n)) / n for j in range(m)]

    Po, pbaro, gto = oracle.core_round(seed, t, m, G)
    assert np.allclose(Po, np.array(P), rtol=1e-13, atol=1e-15)
    assert np.allclose(pbaro, np.array(pbar), rtol=1e-13, atol=1e-15)
    assert np.allclose(gto, np.array(gt), rtol=1e-12, atol=1e-15)
    # single machine: Algorithm 1 verbatim, a~ = (1/m) sum_j <a, xi_j> xi_j
    a = G[0]
    p1 = oracle.project(seed, t, m, a)[0]
    a_t = oracle.reconstruct(seed, t, p1, d)
    want = [sum(sum(float(a[kk]) * xi[j][kk] for kk in range(d)) * xi[j][k] for j in range(m)) / m
            for k in range(d)]
    assert np.allclose(a_t, np.array(want), rtol=1e-12, atol=1e-15)


def test_unit_vector_probes():
    seed, t, d, m = 3, 2, 37, 5          # d not a multiple of 4 on purpose
    for k in (0, 1, 4, 35, 36):
        e = np.zeros((1, d), dtype=np.float32)
        e[0, k] = 1.0
        p = oracle.project(seed, t, m, e)[0]
        for j in range(m):
            assert p[j] == oracle.xi_block(seed, t, j, k >> 2)[k & 3]
    for j in range(m):
        pbar = np.zeros(m)
        pbar[j] = m                       # (1/m) * m * xi_j = xi_j
        assert np.allclose(oracle.reconstruct(seed, t, pbar, d), oracle.xi_range(seed, t, j, 0, d),
                           rtol=1e-15, atol=0)


@pytest.mark.parametrize("d,m,n", [(8, 3, 2), (4096, 16, 4), (1001, 7, 3), (1, 1, 1), (5, 2, 1)])
def test_inner_product_identity_and_linearity(d, m, n):
    seed, t = 1, 4
    G = core_inputs.gradients(n, d, seed=0).numpy()
    P, pbar, gt = oracle.core_round(seed, t, m, G)
    gbar = G.astype(np.float64).mean(axis=0)
    # <gbar, gtilde> = (1/m) sum_j pbar_j^2   (from the estimator's definition)
    assert math.isclose(float(gbar @ gt), float((pbar**2).sum() / m), rel_tol=1e-10, abs_tol=1e-13)
    # reconstruct(mean_i P_i) == mean_i reconstruct(P_i)
    each = np.stack([oracle.reconstruct(seed, t, P[i], d) for i in range(n)])
    assert np.allclose(each.mean(axis=0), gt, rtol=1e-11, atol=1e-13)
    # project(mean_i g_i) == mean_i project(g_i)
    pm = oracle.project(seed, t, m, gbar[None, :])[0]
    assert np.allclose(pm, pbar, rtol=1e-10, atol=1e-12)
    # exact scaling by a power of two
    P2, pbar2, gt2 = oracle.core_round(seed, t, m, (G * np.float32(4.0)))
    assert np.array_equal(P2, 4 * P) and np.array_equal(gt2, 4 * gt)
    # a different round index gives different vectors
    assert not np.allclose(oracle.project(seed, t + 1, m, G), P)


def test_aggregate_is_mean_over_machines():
    P = np.arange(12, dtype=np.float64).reshape(3, 4)
    assert np.array_equal(oracle.aggregate(P), np.array([4.0, 5.0, 6.0, 7.0]))


def test_slices_compose():
    seed, t, d, m = 8, 1, 103, 4
    g = core_inputs.gradients(1, d, seed=5).numpy()[0]
    for j in range(m):
        full = oracle.project_slice(seed, t, j, g, 0, d)
        cuts = [0, 1, 7, 8, 50, 101, d]
        parts = sum(oracle.project_slice(seed, t, j, g, a, b) for a, b in zip(cuts[:-1], cuts[1:]))
        assert math.isclose(full, parts, rel_tol=1e-12, abs_tol=1e-13)
    pbar = np.array([0.3, -1.2, 2.0, 0.5])
    whole = oracle.reconstruct(seed, t, pbar, d)
    for a, b in [(0, 4), (3, 9), (5, 6), (98, 103), (0, d)]:
        assert np.array_equal(oracle.reconstruct_slice(seed, t, pbar, a, b), whole[a:b])


def test_bf16_inputs_are_widened_exactly():
    seed, t, d, m, n = 2, 0, 257, 3, 2
    Gb = core_inputs.gradients(n, d, seed=1, dist="student_t3", dtype="bf16")
    bits = core_inputs.to_oracle_array(Gb)
    assert bits.dtype == np.uint16
    widened = Gb.float().numpy()
    assert np.array_equal(oracle.project(seed, t, m, bits), oracle.project(seed, t, m, widened))


def test_estimator_moments_over_seeds():
    # Lemma 3.1 (unbiased) and the exact second moment from the proof of Lemma 3.2 at A = I
    d, S = 64, 4000
    a = core_inputs.gradients(1, d, seed=3).numpy()
    a2 = float((a.astype(np.float64) ** 2).sum())
    for m in (4, 16):
        acc = np.zeros(d)
        sq = np.zeros(S)
        for s in range(S):
            _, _, gt = oracle.core_round(1000 + s, 0, m, a)
            acc += gt
            sq[s] = (gt**2).sum()
        mean = acc / S
        # E||mean - a||^2 = (d+1) ||a||^2 / (m S)
        ratio = float(((mean - a[0]) ** 2).sum()) / ((d + 1) * a2 / (m * S))
        assert 0.6 < ratio < 1.5
        want = (d + m + 1) / m * a2
        se = sq.std(ddof=1) / math.sqrt(S)
        assert abs(sq.mean() - want) < 4 * se
        assert se < 0.05 * want


def test_messages_are_gaussian_with_norm_of_a():
    # p = Xi a ~ N(0, ||a||^2 I_m)
    d, m = 256, 2048
    a = core_inputs.gradients(1, d, seed=9).numpy()
    norm = math.sqrt(float((a.astype(np.float64) ** 2).sum()))
    p = oracle.project(77, 0, m, a)[0] / norm
    assert stats.kstest(p, "norm").pvalue > 1e-3
    assert abs((p**2).mean() - 1) < 4 * math.sqrt(2 / m)


def test_round_on_tiny_workload_runs_and_reduces_error_with_m():
    w = core_inputs.WORKLOADS["tiny"]
    G = core_inputs.workload_gradients("tiny", seed=0).numpy()
    gbar = G.astype(np.float64).mean(axis=0)
    errs = []
    for m in (16, 256):
        _, _, gt = oracle.core_round(1, 0, m, G)
        errs.append(float(((gt - gbar) ** 2).sum() / (gbar**2).sum()))
    # relative error ~ (d+1)/m
    assert 0.5 * (w.d + 1) / 16 < errs[0] < 2 * (w.d + 1) / 16
    assert 0.6 * (w.d + 1) / 256 < errs[1] < 1.6 * (w.d + 1) / 256
