"""Pins for the oracle's decentralised variant (Algorithm 5: gossip averaging of the messages), CPU only.

What fixes the expectations: a three-machine round worked by hand, numpy's matrix power, the spectrum of
the gossip matrix (limit = the centralised mean, error contracting at the second largest eigenvalue
modulus), conservation of the mean by a doubly stochastic matrix, and the centralised iteration of
Algorithm 2 (pinned on its own) as the limit of many gossip rounds.
"""
import math

import numpy as np

import core_inputs
import oracle


def problem(seed=11, n=4):
    ls = core_inputs.least_squares(n=n, rows=40, d=48, seed=seed, decay=1.0, noise=0.05)
    return ls.A.numpy(), ls.b.numpy()


def test_one_round_by_hand():
    # three machines in a line 0 - 1 - 2 with weights chosen by hand (not from the generator)
    W = np.array([[0.75, 0.25, 0.0], [0.25, 0.5, 0.25], [0.0, 0.25, 0.75]])
    P = np.array([[4.0, 0.0], [0.0, 8.0], [-4.0, 4.0]])
    want = np.array([[3.0, 2.0], [0.0, 5.0], [-3.0, 5.0]])
    assert np.array_equal(oracle.gossip_round(W, P), want)
    assert np.array_equal(oracle.gossip_average(W, P, 1), want)
    assert np.array_equal(oracle.gossip_average(W, P, 0), P)
    # transposing W would not show here (symmetric): an asymmetric row-stochastic matrix tells rows from columns
    Wa = np.array([[1.0, 0.0], [0.5, 0.5]])
    assert np.array_equal(oracle.gossip_round(Wa, np.array([[2.0], [6.0]])), np.array([[2.0], [4.0]]))


def test_many_rounds_are_a_matrix_power_and_reach_the_mean():
    rng = np.random.default_rng(1)
    for topology, n in [("ring", 8), ("torus", 12), ("ring", 5), ("torus", 16), ("complete", 6)]:
        W = core_inputs.gossip_matrix(topology, n)
        P = rng.standard_normal((n, 7))
        mean = P.mean(axis=0)
        for rounds in (1, 3, 10):
            assert np.allclose(oracle.gossip_average(W, P, rounds), np.linalg.matrix_power(W, rounds) @ P,
                               rtol=1e-12, atol=1e-14)
            # a doubly stochastic matrix conserves the network mean at every round
            assert np.allclose(oracle.gossip_average(W, P, rounds).mean(axis=0), mean, rtol=0, atol=1e-14)
        far = oracle.gossip_average(W, P, 2000)
        assert np.allclose(far, np.tile(mean, (n, 1)), rtol=0, atol=1e-12)
    one = oracle.gossip_average(core_inputs.gossip_matrix("complete", 6), P[:6], 1)
    assert np.allclose(one, np.tile(P[:6].mean(axis=0), (6, 1)), atol=1e-15)


def test_error_contracts_at_the_second_eigenvalue():
    rng = np.random.default_rng(2)
    for topology, n in [("ring", 8), ("torus", 16), ("ring", 16)]:
        W = core_inputs.gossip_matrix(topology, n)
        lam = np.sort(np.abs(np.linalg.eigvalsh(W)))[::-1]
        assert math.isclose(lam[0], 1.0, rel_tol=1e-12) and lam[1] < 1.0
        P = rng.standard_normal((n, 5))
        mean = np.tile(P.mean(axis=0), (n, 1))
        e0 = np.linalg.norm(P - mean)
        prev = e0
        for rounds in range(1, 40):
            e = np.linalg.norm(oracle.gossip_average(W, P, rounds) - mean)
            assert e <= lam[1] ** rounds * e0 * (1 + 1e-9)          # the bound behind the 1/sqrt(gamma) cost
            assert e <= prev * (1 + 1e-12)
            prev = e
        # the asymptotic rate is the second eigenvalue itself
        e_a = np.linalg.norm(oracle.gossip_average(W, P, 60) - mean)
        e_b = np.linalg.norm(oracle.gossip_average(W, P, 61) - mean)
        assert math.isclose(e_b / e_a, lam[1], rel_tol=1e-3)


def test_decentralised_step_tends_to_the_centralised_step():
    A, b = problem(n=4)
    n, rows, d = A.shape
    m, seed, t, h = 6, 4, 2, 0.3
    rng = np.random.default_rng(0)
    x = rng.standard_normal(d)
    central = oracle.gd_step(seed, t, m, A, b, h, x)
    W = core_inputs.gossip_matrix("ring", n)
    x_many, spread_many = oracle.decentralized_step(seed, t, m, A, b, W, 400, h, x)
    assert np.allclose(x_many, central, rtol=0, atol=1e-12) and spread_many < 1e-12
    # the complete graph reaches the mean in one round, from any reader
    Wc = core_inputs.gossip_matrix("complete", n)
    for reader in range(n):
        x_c, spread = oracle.decentralized_step(seed, t, m, A, b, Wc, 1, h, x, reader=reader)
        assert np.allclose(x_c, central, rtol=0, atol=1e-13) and spread < 1e-13
    # the printed n/m prefactor is the sum convention: n times the step of the mean convention
    x_printed, _ = oracle.decentralized_step(seed, t, m, A, b, W, 400, h / n, x, as_printed=True)
    assert np.allclose(x_printed, central, rtol=0, atol=1e-12)
    # no gossip at all: the reader reconstructs from its own message only (a one-machine round)
    x_none, spread_none = oracle.decentralized_step(seed, t, m, A, b, W, 0, h, x, reader=2)
    G = oracle.ls_grad(A, b, x)
    own = oracle.reconstruct(seed, t, oracle.project(seed, t, m, G[2:3])[0], d)
    assert np.allclose(x_none, x - h * own, rtol=0, atol=1e-13) and spread_none > 0
    # few rounds: the distance to the centralised iterate shrinks with the rounds
    errs = [np.linalg.norm(oracle.decentralized_step(seed, t, m, A, b, W, r, h, x)[0] - central) for r in (0, 2, 6, 20)]
    assert errs[0] > errs[1] > errs[2] > errs[3]


def test_spread_is_the_largest_deviation_from_the_reader():
    A, b = problem(n=4)
    m, seed, t = 5, 9, 0
    x = np.linspace(-1, 1, 48)
    W = core_inputs.gossip_matrix("ring", 4)
    G = oracle.ls_grad(A, b, x)
    P = oracle.gossip_average(W, oracle.project(seed, t, m, G), 3)
    for reader in (0, 3):
        _, spread = oracle.decentralized_step(seed, t, m, A, b, W, 3, 0.1, x, reader=reader)
        assert math.isclose(spread, float(np.abs(P - P[reader]).max()), rel_tol=1e-13)


def test_gossip_matrices_are_valid_networks():
    for topology in ("ring", "torus", "complete"):
        for n in (1, 2, 3, 4, 8, 9, 12, 16):
            W = core_inputs.gossip_matrix(topology, n)
            assert np.allclose(W, W.T) and np.allclose(W.sum(axis=1), 1.0) and (W >= 0).all()
    W = core_inputs.gossip_matrix("ring", 8)
    assert W[0, 1] > 0 and W[0, 7] > 0 and W[0, 2] == 0 and W[0, 4] == 0
    W = core_inputs.gossip_matrix("torus", 16)               # 4 x 4 grid: 0's neighbours are 1, 3, 4, 12
    assert {int(l) for l in np.nonzero(W[0])[0]} == {0, 1, 3, 4, 12}
