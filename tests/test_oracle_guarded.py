"""Pins for the oracle's Algorithm-3 step (CORE-GD with the comparison step), CPU only.

What fixes the expectations: the definition (trial point from the round primitives, argmin over two
points with ties kept), monotonicity of f along any trajectory, and the behaviour at the two extremes of
the step size (a tiny step is accepted whenever the estimate correlates with the gradient; a huge step
is rejected).
"""
import numpy as np

import core_inputs
import oracle


def problem(seed=11):
    ls = core_inputs.least_squares(n=3, rows=40, d=48, seed=seed, decay=1.0, noise=0.05)
    return ls.A.numpy(), ls.b.numpy()


def test_definition_from_the_primitives():
    A, b = problem()
    d, m, seed, t, h = 48, 6, 4, 2, 0.3
    rng = np.random.default_rng(0)
    x = rng.standard_normal(d)
    f0 = oracle.ls_loss(A, b, x)
    trial = oracle.gd_step(seed, t, m, A, b, h, x)
    f_trial = oracle.ls_loss(A, b, trial)
    kept, f_kept, accepted = oracle.gd_step_guarded(seed, t, m, A, b, h, x, f0)
    if f_trial < f0:
        assert accepted and np.array_equal(kept, trial) and f_kept == f_trial
    else:
        assert not accepted and np.array_equal(kept, x) and f_kept == f0


def test_loss_never_increases_and_both_branches_occur():
    A, b = problem()
    d, m = 48, 2
    L = core_inputs.lipschitz_constant(core_inputs.least_squares(n=3, rows=40, d=48, seed=11, decay=1.0,
                                                                 noise=0.05).A)
    x = np.zeros(d)
    f = oracle.ls_loss(A, b, x)
    outcomes = []
    for k in range(120):
        x, f_new, acc = oracle.gd_step_guarded(1, k, m, A, b, 0.7 / L, x, f)   # too long for m=2: some rejections
        assert f_new <= f
        assert abs(f_new - oracle.ls_loss(A, b, x)) <= 1e-12 * max(1.0, f_new)
        f = f_new
        outcomes.append(acc)
    assert any(outcomes) and not all(outcomes)
    assert f < 0.7 * oracle.ls_loss(A, b, np.zeros(d))


def test_huge_step_is_rejected_and_keeps_the_point():
    A, b = problem()
    rng = np.random.default_rng(3)
    x = rng.standard_normal(48)
    f0 = oracle.ls_loss(A, b, x)
    kept, f_kept, acc = oracle.gd_step_guarded(2, 0, 4, A, b, 1e6, x, f0)
    assert not acc and np.array_equal(kept, x) and f_kept == f0


def test_tie_keeps_the_current_point():
    A, b = problem()
    x = np.linspace(-1, 1, 48)
    f0 = oracle.ls_loss(A, b, x)
    kept, f_kept, acc = oracle.gd_step_guarded(2, 0, 4, A, b, 0.0, x, f0)      # h = 0: trial == x, f equal
    assert not acc and np.array_equal(kept, x) and f_kept == f0
