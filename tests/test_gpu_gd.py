"""GPU parity of the least-squares CORE-GD driver (Algorithm 2) against the oracle.

The two sides run their own trajectories from x0 = 0 with the same inputs, step and round
indices t = k.  Bars: machine gradients relative L2 <= 1e-5; iterates and losses within
1e-3 relative along the whole trajectory (errors pass through a map that does not expand
in expectation; the paper states no tolerance for trajectories).
"""
import numpy as np
import pytest
import torch

import core_inputs
import oracle
from helpers import rel_l2

pytestmark = pytest.mark.gpu

TRAJ_TOL = 1e-3


@pytest.fixture(scope="module")
def core_mod():
    import paper_2309_13307_b200 as core_mod
    core_mod.lib()
    return core_mod


def run_both(core_mod, ls_in, m, iters, seed=1):
    A, b = ls_in.A, ls_in.b
    n, rows, d = A.shape
    L = core_inputs.lipschitz_constant(A)
    h = float(np.float32(1.0 / L))                 # rounded once, given to both sides
    Ah, bh = A.cpu().numpy(), b.cpu().numpy()

    ctx = core_mod.Core(seed, d, m)
    ls = core_mod.LeastSquares(A, b)
    x = torch.zeros(d, dtype=torch.float32, device="cuda")
    xo = np.zeros(d)

    # machine gradients at a non-trivial point
    xp = core_inputs.gradients(1, d, seed=21, device="cuda")[0].contiguous()
    G = ctx.core_ls_gradients(ls, xp).cpu().numpy()
    Go = oracle.ls_grad(Ah, bh, xp.cpu().numpy().astype(np.float64))
    for i in range(n):
        assert rel_l2(G[i], Go[i]) <= 1e-5

    gpu_loss = [float(ctx.core_ls_loss(ls, x).item())]
    orc_loss = [oracle.ls_loss(Ah, bh, xo)]
    for k in range(iters):
        assert ctx.core_get_round() == k
        ctx.core_gd_step(ls, h, x)
        xo = oracle.gd_step(seed, k, m, Ah, bh, h, xo)
        gpu_loss.append(float(ctx.core_ls_loss(ls, x).item()))
        orc_loss.append(oracle.ls_loss(Ah, bh, xo))
        assert rel_l2(x.cpu().numpy(), xo) <= TRAJ_TOL, k
    gpu_loss, orc_loss = np.array(gpu_loss), np.array(orc_loss)
    assert (np.abs(gpu_loss - orc_loss) <= TRAJ_TOL * orc_loss).all()
    return gpu_loss, orc_loss


@pytest.mark.parametrize("n,rows,d,m,iters", [(2, 64, 128, 16, 40), (3, 50, 1001, 8, 20), (8, 128, 4096, 64, 10)])
def test_small_problems(core_mod, n, rows, d, m, iters):
    ls_in = core_inputs.least_squares(n=n, rows=rows, d=d, seed=0, device="cuda")
    gpu_loss, _ = run_both(core_mod, ls_in, m, iters)
    assert gpu_loss[-1] < gpu_loss[0]


def test_least_squares_workload_200_iterations(core_mod):
    # n=8 machines, A_i 2048 x 8192, power-law spectrum, m=64, step 1/L, 200 iterations
    ls_in = core_inputs.least_squares(n=8, rows=2048, d=8192, seed=0, device="cuda")
    gpu_loss, orc_loss = run_both(core_mod, ls_in, 64, 200)
    assert gpu_loss[-1] < 0.5 * gpu_loss[0]


@pytest.mark.parametrize("n,rows,d,m", [(8, 256, 4096, 64), (3, 50, 1001, 8)])
def test_step_equals_its_parts(core_mod, n, rows, d, m):
    """core_gd_step never stores the machine gradients (where the single-pass gradient kernel applies the
    projection adds their partial sums while it stages its tiles).  Building the same step from the entry
    points that do store them - gradients, round, update - must give the same iterate: the sums are the same
    and taken in the same order, so only the final multiply-add may round differently."""
    ls_in = core_inputs.least_squares(n=n, rows=rows, d=d, seed=3, device="cuda")
    h = 0.37
    x0 = core_inputs.gradients(1, d, seed=5, device="cuda")[0].contiguous()
    ls = core_mod.LeastSquares(ls_in.A, ls_in.b)
    whole, parts = core_mod.Core(9, d, m), core_mod.Core(9, d, m)
    whole.core_set_round(4)
    parts.core_set_round(4)
    x = x0.clone()
    whole.core_gd_step(ls, h, x)
    G = parts.core_ls_gradients(ls, x0)
    _, gt = parts.core_round(G)
    want = x0.double() - h * gt.double()
    assert whole.core_get_round() == parts.core_get_round() == 5
    err = (x.double() - want).abs().max().item()
    assert err <= 2e-7 * max(1.0, want.abs().max().item()), err
