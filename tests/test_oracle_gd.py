"""Pins for the oracle's least-squares CORE-GD driver (Algorithm 2), CPU only.

Expected values come from linear algebra done with numpy on the explicit Hessian
(closed-form gradient-descent recursion, exact expected decrease from
E[xi xi^T H xi xi^T] = tr(H) I + 2H in the proof of Lemma 3.2) and from
Theorem 4.2's contraction factor 1 - 3 m mu / (16 tr A).
"""
import math

import numpy as np

import core_inputs
import oracle


def small_problem(n=2, rows=48, d=32, seed=4):
    ls = core_inputs.least_squares(n=n, rows=rows, d=d, seed=seed, decay=0.5, noise=0.05)
    A = ls.A.numpy()
    b = ls.b.numpy()
    A64 = A.astype(np.float64)
    H = sum(A64[i].T @ A64[i] for i in range(n)) / (n * rows)
    c = sum(A64[i].T @ b[i].astype(np.float64) for i in range(n)) / (n * rows)
    x_opt = np.linalg.solve(H, c)
    return A, b, H, c, x_opt


def f_numpy(A, b, x):
    n, rows, _ = A.shape
    return sum(((A[i].astype(np.float64) @ x - b[i]) ** 2).sum() / (2 * rows) for i in range(n)) / n


def test_loss_and_gradient_against_numpy_and_finite_differences():
    A, b, H, c, _ = small_problem()
    rng = np.random.default_rng(0)
    x = rng.standard_normal(A.shape[2])
    assert math.isclose(oracle.ls_loss(A, b, x), f_numpy(A, b, x), rel_tol=1e-12)
    G = oracle.ls_grad(A, b, x)
    # mean of the machine gradients is the gradient of f: H x - c
    assert np.allclose(G.mean(axis=0), H @ x - c, rtol=1e-10, atol=1e-13)
    # machine i's gradient by central differences of f_i
    i, eps = 1, 1e-6
    for k in (0, 7, 31):
        e = np.zeros_like(x)
        e[k] = eps
        fi = lambda y: ((A[i].astype(np.float64) @ y - b[i]) ** 2).sum() / (2 * A.shape[1])
        assert math.isclose(G[i, k], (fi(x + e) - fi(x - e)) / (2 * eps), rel_tol=1e-6, abs_tol=1e-9)


def test_exact_gradient_limit_follows_closed_form_recursion():
    A, b, H, c, x_opt = small_problem()
    d = A.shape[2]
    L = np.linalg.eigvalsh(H)[-1]
    h = 1.0 / L
    x = np.zeros(d)
    for k in range(25):
        x = oracle.gd_step(1, k, 4, A, b, h, x, exact=True)
    M = np.linalg.matrix_power(np.eye(d) - h * H, 25)
    assert np.allclose(x - x_opt, M @ (np.zeros(d) - x_opt), rtol=1e-9, atol=1e-12)


def test_one_step_is_x_minus_h_gtilde():
    A, b, H, c, _ = small_problem()
    d, m, seed, t = A.shape[2], 6, 21, 3
    rng = np.random.default_rng(1)
    x = rng.standard_normal(d)
    G = oracle.ls_grad(A, b, x)
    _, _, gt = oracle.core_round(seed, t, m, G)
    x1 = oracle.gd_step(seed, t, m, A, b, 0.37, x)
    assert np.allclose(x1, x - 0.37 * gt, rtol=1e-13, atol=1e-15)


def test_expected_decrease_matches_exact_second_moment():
    # E f(x+) = f - h |g|^2 + (h^2/2) [ (1/m)(tr(H)|g|^2 + 2 g^T H g) + (1 - 1/m) g^T H g ]
    A, b, H, c, _ = small_problem()
    d, m, S = A.shape[2], 4, 3000
    rng = np.random.default_rng(2)
    x = rng.standard_normal(d)
    g = H @ x - c
    h = m / (4 * np.trace(H))
    f0 = f_numpy(A, b, x)
    gHg = g @ H @ g
    want = f0 - h * (g @ g) + 0.5 * h * h * ((np.trace(H) * (g @ g) + 2 * gHg) / m + (1 - 1 / m) * gHg)
    vals = np.array([f_numpy(A, b, oracle.gd_step(500 + s, 0, m, A, b, h, x)) for s in range(S)])
    se = vals.std(ddof=1) / math.sqrt(S)
    assert abs(vals.mean() - want) < 4 * se
    assert se < 0.02 * abs(f0 - want)      # the test resolves the decrease itself


def test_theorem_4_2_contraction():
    # h = m / (4 tr A), m <= tr(A)/L with A = H: E f(x+) - f* <= (1 - 3 m mu / (16 tr A)) (f(x) - f*)
    A, b, H, c, x_opt = small_problem()
    d = A.shape[2]
    ev = np.linalg.eigvalsh(H)
    mu, L, tr = ev[0], ev[-1], ev.sum()
    m = int(tr / L)
    assert m >= 2
    h = m / (4 * tr)
    fstar = f_numpy(A, b, x_opt)
    rng = np.random.default_rng(3)
    x = x_opt + rng.standard_normal(d)
    S = 1500
    vals = np.array([f_numpy(A, b, oracle.gd_step(9000 + s, 0, m, A, b, h, x)) for s in range(S)])
    ratio = (vals.mean() - fstar) / (f_numpy(A, b, x) - fstar)
    se = vals.std(ddof=1) / math.sqrt(S) / (f_numpy(A, b, x) - fstar)
    assert ratio - 4 * se <= 1 - 3 * m * mu / (16 * tr)
    assert ratio < 1.0


def test_trajectory_descends_on_small_power_law_problem():
    # step 1/L outside the theorem's regime (m > tr/L), as in the least-squares workload
    ls = core_inputs.least_squares(n=2, rows=64, d=128, seed=0)
    A, b = ls.A.numpy(), ls.b.numpy()
    L = core_inputs.lipschitz_constant(ls.A)
    x = np.zeros(128)
    losses = [oracle.ls_loss(A, b, x)]
    for k in range(60):
        x = oracle.gd_step(1, k, 16, A, b, 1.0 / L, x)
        losses.append(oracle.ls_loss(A, b, x))
    assert losses[-1] < 0.5 * losses[0]
