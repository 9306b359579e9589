"""Pins for the oracle's CORE-AGD step (Algorithm 4: heavy ball with the CORE estimate), CPU only.

Expected values: the heavy-ball recursion on a quadratic written as a 2d x 2d linear map (numpy), the
definition of one step from the round primitives, unbiasedness of the step (Lemma 3.1), and faster
convergence than plain gradient descent on an ill-conditioned quadratic in the exact-gradient limit.
"""
import math

import numpy as np

import core_inputs
import oracle


def problem(n=2, rows=64, d=24, seed=7, decay=1.0):
    ls = core_inputs.least_squares(n=n, rows=rows, d=d, seed=seed, decay=decay, noise=0.02)
    A, b = ls.A.numpy(), ls.b.numpy()
    A64 = A.astype(np.float64)
    H = sum(A64[i].T @ A64[i] for i in range(n)) / (n * rows)
    c = sum(A64[i].T @ b[i].astype(np.float64) for i in range(n)) / (n * rows)
    return A, b, H, c, np.linalg.solve(H, c)


def test_exact_limit_is_the_heavy_ball_linear_map():
    A, b, H, c, x_opt = problem()
    d = H.shape[0]
    ev = np.linalg.eigvalsh(H)
    h = 1.0 / ev[-1]
    beta = math.sqrt(h * ev[0])
    g = 1.0 - beta
    # e_{k+1} = (1+g)(I - hH) e_k - g (I - hH) e_{k-1},  e = x - x*
    T = np.eye(d) - h * H
    M = np.block([[(1 + g) * T, -g * T], [np.eye(d), np.zeros((d, d))]])
    rng = np.random.default_rng(0)
    x0 = rng.standard_normal(d)
    x, xp = x0.copy(), x0.copy()                       # x^{-1} = x^0
    for k in range(30):
        x, xp = oracle.agd_step(1, k, 4, A, b, h, beta, x, xp, exact=True)
    want = np.linalg.matrix_power(M, 30) @ np.concatenate([x0 - x_opt, x0 - x_opt])
    assert np.allclose(x - x_opt, want[:d], rtol=1e-8, atol=1e-12)
    assert np.allclose(xp - x_opt, want[d:], rtol=1e-8, atol=1e-12)


def test_one_step_from_the_round_primitives():
    A, b, H, c, _ = problem()
    d, m, seed, t, h, beta = H.shape[0], 5, 3, 9, 0.4, 0.25
    rng = np.random.default_rng(1)
    x, xp = rng.standard_normal(d), rng.standard_normal(d)
    y = x + (1 - beta) * (x - xp)
    _, _, gt = oracle.core_round(seed, t, m, oracle.ls_grad(A, b, y))
    x1, xp1 = oracle.agd_step(seed, t, m, A, b, h, beta, x, xp)
    assert np.allclose(x1, y - h * gt, rtol=1e-13, atol=1e-15)
    assert np.array_equal(xp1, x)
    # beta = 1 removes the momentum: the step is then a CORE-GD step from x
    x2, _ = oracle.agd_step(seed, t, m, A, b, h, 1.0, x, xp)
    assert np.allclose(x2, oracle.gd_step(seed, t, m, A, b, h, x), rtol=1e-13, atol=1e-15)


def test_step_is_unbiased_around_the_exact_heavy_ball_step():
    A, b, H, c, _ = problem()
    d, m, h, beta, S = H.shape[0], 4, 0.5, 0.3, 3000
    rng = np.random.default_rng(2)
    x, xp = rng.standard_normal(d), rng.standard_normal(d)
    exact, _ = oracle.agd_step(0, 0, m, A, b, h, beta, x, xp, exact=True)
    acc = np.zeros(d)
    sq = 0.0
    for s in range(S):
        xs, _ = oracle.agd_step(100 + s, 0, m, A, b, h, beta, x, xp)
        acc += xs
        sq += float(((xs - exact) ** 2).sum())
    # the mean over seeds approaches the exact step at the Monte-Carlo rate
    assert float(((acc / S - exact) ** 2).sum()) < 16 * (sq / S) / S


def test_momentum_beats_plain_descent_on_an_ill_conditioned_quadratic():
    A, b, H, c, x_opt = problem(d=32, rows=96, decay=2.5)
    ev = np.linalg.eigvalsh(H)
    h = 1.0 / ev[-1]
    beta = math.sqrt(h * ev[0])
    d = H.shape[0]
    xg = np.zeros(d)
    xa, xap = np.zeros(d), np.zeros(d)
    for k in range(400):
        xg = oracle.gd_step(1, k, 4, A, b, h, xg, exact=True)
        xa, xap = oracle.agd_step(1, k, 4, A, b, h, beta, xa, xap, exact=True)
    f = lambda x: oracle.ls_loss(A, b, x) - oracle.ls_loss(A, b, x_opt)
    assert f(xa) < 0.1 * f(xg)
