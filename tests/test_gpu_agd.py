"""GPU parity of the CORE-AGD step (Algorithm 4) and of the fused update of the GD step.

Both sides run their own trajectories from x0 = x_prev = 0 with the same inputs, step, momentum and
round indices.  Bar: iterate relative L2 <= 1e-3 along the trajectory (as for the GD driver).
"""
import math

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


@pytest.mark.parametrize("n,rows,d,m,iters", [(2, 64, 128, 16, 40), (3, 50, 1001, 8, 25), (8, 256, 8192, 64, 12)])
def test_agd_trajectory(core_mod, n, rows, d, m, iters):
    ls_in = core_inputs.least_squares(n=n, rows=rows, d=d, seed=2, device="cuda")
    A, b = ls_in.A, ls_in.b
    L = core_inputs.lipschitz_constant(A, iters=60)
    h = float(np.float32(0.5 / L))
    beta = float(np.float32(0.2))
    Ah, bh = A.cpu().numpy(), b.cpu().numpy()
    ctx = core_mod.Core(5, d, m)
    ls = core_mod.LeastSquares(A, b)
    x = torch.zeros(d, dtype=torch.float32, device="cuda")
    xp = torch.zeros(d, dtype=torch.float32, device="cuda")
    xo, xpo = np.zeros(d), np.zeros(d)
    for k in range(iters):
        assert ctx.core_get_round() == k
        ctx.core_agd_step(ls, h, beta, x, xp)
        xo, xpo = oracle.agd_step(5, k, m, Ah, bh, h, beta, xo, xpo)
        assert rel_l2(x.cpu().numpy(), xo) <= TRAJ_TOL, k
        assert rel_l2(xp.cpu().numpy(), xpo) <= TRAJ_TOL or k == 0, k
    f0 = oracle.ls_loss(Ah, bh, np.zeros(d))
    assert float(ctx.core_ls_loss(ls, x).item()) < f0


def test_agd_with_unit_beta_is_the_gd_step(core_mod):
    ls_in = core_inputs.least_squares(n=2, rows=40, d=515, seed=3, device="cuda")
    ctx_a = core_mod.Core(9, 515, 4)
    ctx_g = core_mod.Core(9, 515, 4)
    ls = core_mod.LeastSquares(ls_in.A, ls_in.b)
    xa = core_inputs.gradients(1, 515, seed=1, device="cuda")[0].contiguous()
    xg = xa.clone()
    xp = core_inputs.gradients(1, 515, seed=2, device="cuda")[0].contiguous()
    x_before = xa.clone()
    ctx_a.core_agd_step(ls, 0.3, 1.0, xa, xp)           # beta = 1: no momentum
    ctx_g.core_gd_step(ls, 0.3, xg)
    assert torch.equal(xa, xg)
    assert torch.equal(xp, x_before)                     # x_prev <- x


def test_gd_step_equals_round_then_update(core_mod):
    """The fused update inside the reconstruction gives x - h * gtilde of the unfused calls."""
    ls_in = core_inputs.least_squares(n=4, rows=32, d=4099, seed=5, device="cuda")
    d, m, h = 4099, 16, 0.25
    ctx = core_mod.Core(3, d, m)
    ls = core_mod.LeastSquares(ls_in.A, ls_in.b)
    x = core_inputs.gradients(1, d, seed=8, device="cuda")[0].contiguous()
    G = ctx.core_ls_gradients(ls, x)
    _, gt = ctx.core_round(G)
    want = torch.addcmul(x, gt, torch.tensor(-h, device="cuda"))
    ctx.core_set_round(0)
    ctx.core_gd_step(ls, h, x)
    assert float((x - want).abs().max()) <= 2e-7 * float(want.abs().max()) + 1e-12
