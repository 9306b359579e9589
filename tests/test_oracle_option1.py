"""Pins for the oracle's Algorithm-3 step with Option I (the step chosen from the size of the combined
messages), CPU only.

The statistic is a reading of a garbled line of the algorithm: p = sqrt((1/m) sum_j pbar_j^2).  What fixes
the expectations here is not the oracle: the law of the messages (a vector a is sent as N(0, ||a||^2 I_m),
so m p^2 / ||gbar||^2 is chi-square with m degrees of freedom), the closed form of the step written out
with the math module, and the definition of the iteration from primitives that are pinned elsewhere.
"""
import math

import numpy as np
from scipy import stats

import core_inputs
import oracle


def problem(seed=11):
    ls = core_inputs.least_squares(n=3, rows=40, d=48, seed=seed, decay=1.0, noise=0.05)
    return ls.A.numpy(), ls.b.numpy()


def test_message_norm_by_hand():
    assert oracle.message_norm(np.array([3.0, -4.0])) == math.sqrt(12.5)
    assert oracle.message_norm(np.array([0.0, 0.0, 0.0])) == 0.0
    assert oracle.message_norm(np.array([-2.0])) == 2.0
    v = np.array([1.0, 2.0, 3.0, 4.0])
    assert math.isclose(oracle.message_norm(v), math.sqrt(30.0 / 4.0), rel_tol=1e-15)
    # scaling the gradients scales the statistic; the sign of a message does not matter
    assert math.isclose(oracle.message_norm(-3.0 * v), 3.0 * oracle.message_norm(v), rel_tol=1e-15)


def test_statistic_squared_estimates_the_squared_gradient_norm():
    """E p^2 = ||gbar||^2 with m p^2 / ||gbar||^2 ~ chi-square(m): mean, spread and the whole law."""
    d, n, m, S = 64, 3, 16, 3000
    G = core_inputs.gradients(n, d, seed=5, dist="scaled_normal").numpy()
    gbar_sq = float((G.astype(np.float64).mean(axis=0) ** 2).sum())
    ratios = np.empty(S)
    for s in range(S):
        pbar = oracle.aggregate(oracle.project(1000 + s, 0, m, G))
        ratios[s] = oracle.message_norm(pbar) ** 2 / gbar_sq
    se = math.sqrt(2.0 / m / S)                                # Var(chi2_m / m) = 2 / m
    assert abs(ratios.mean() - 1.0) < 4 * se
    assert abs(ratios.var() - 2.0 / m) < 0.2 * (2.0 / m)
    assert stats.kstest(ratios * m, "chi2", args=(m,)).pvalue > 1e-3


def test_statistic_concentrates_as_m_grows():
    d, n = 64, 2
    G = core_inputs.gradients(n, d, seed=6).numpy()
    gbar = math.sqrt(float((G.astype(np.float64).mean(axis=0) ** 2).sum()))
    spread = {}
    for m in (4, 64, 1024):
        r = [oracle.message_norm(oracle.aggregate(oracle.project(50 + s, 1, m, G))) / gbar for s in range(40)]
        spread[m] = float(np.std(r))
        assert abs(np.mean(r) - 1.0) < 4 * (1 / math.sqrt(2 * m)) / math.sqrt(40) + 1.0 / (4 * m)
    assert spread[1024] < spread[64] < spread[4]
    assert spread[1024] < 2.0 / math.sqrt(2 * 1024)


def test_step_rule_closed_form_both_branches():
    m, d, r1, H, c = 16, 4096, 3.0, 2.5, 1.0 / 1600.0
    first = m / (16 * r1)
    for p in (1e-12, 1e-3, 0.7, 5.0, 1e6):
        second = c / math.sqrt(H) / math.sqrt(p) * d ** -0.75 * m ** 0.75
        assert math.isclose(oracle.option1_step(p, m, d, r1, H, c), min(first, second), rel_tol=1e-13)
    # a vanishing gradient selects the first term, a large one the second
    assert oracle.option1_step(0.0, m, d, r1, H, c) == first
    assert oracle.option1_step(1e-30, m, d, r1, H, c) == first
    assert oracle.option1_step(1e6, m, d, r1, H, c) < first
    # monotone: a larger statistic never lengthens the step
    hs = [oracle.option1_step(p, m, d, r1, H, c) for p in np.logspace(-6, 6, 40)]
    assert all(a >= b for a, b in zip(hs, hs[1:]))
    # default constant is the printed 1/1600
    assert oracle.option1_step(2.0, m, d, r1, H) == oracle.option1_step(2.0, m, d, r1, H, 1.0 / 1600.0)


def test_iteration_is_its_definition_from_the_primitives():
    A, b = problem()
    n, rows, d = A.shape
    m, seed, t = 6, 4, 2
    r1, H, c = 0.8, 0.05, 3.0
    rng = np.random.default_rng(0)
    x = rng.standard_normal(d)
    f0 = oracle.ls_loss(A, b, x)
    kept, f_kept, accepted, p, h = oracle.gd_step_option1(seed, t, m, A, b, r1, H, c, x, f0)
    # the statistic is that of this round's combined messages, the step its closed form
    G = oracle.ls_grad(A, b, x)
    pbar = oracle.aggregate(oracle.project(seed, t, m, G))
    assert p == oracle.message_norm(pbar)
    assert math.isclose(p, math.sqrt(float((pbar ** 2).sum()) / m), rel_tol=1e-14)
    want_h = min(m / (16 * r1), c / math.sqrt(H) / math.sqrt(p) * d ** -0.75 * m ** 0.75)
    assert math.isclose(h, want_h, rel_tol=1e-13)
    # with that step the iteration is the caller-fixed-step iteration (pinned on its own)
    kept2, f2, acc2 = oracle.gd_step_guarded(seed, t, m, A, b, h, x, f0)
    assert accepted == acc2 and np.array_equal(kept, kept2) and f_kept == f2


def test_loss_never_increases_and_the_step_adapts():
    A, b = problem()
    d, m = 48, 4
    x = np.zeros(d)
    f = oracle.ls_loss(A, b, x)
    steps, stats_p = [], []
    for k in range(60):
        x, f_new, acc, p, h = oracle.gd_step_option1(3, k, m, A, b, 0.1, 1.0, 1.0, x, f)
        assert f_new <= f
        f = f_new
        steps.append(h)
        stats_p.append(p)
    assert f < 0.8 * oracle.ls_loss(A, b, np.zeros(d))
    # as the gradient (hence p) shrinks the second term grows: steps at the end are not shorter
    assert np.mean(stats_p[-10:]) < np.mean(stats_p[:10])
    assert np.mean(steps[-10:]) >= np.mean(steps[:10])
