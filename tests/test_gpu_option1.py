"""GPU parity of Algorithm 3 with Option I (step chosen on the device from the combined messages).

Both sides run their own trajectories.  Per iteration: the statistic p and the step h agree to 1e-4
relative (p is a smooth function of the messages, themselves within 1e-4 ||g||); the accept/reject
decision agrees wherever the oracle's margin is far above the fp32-vs-fp64 difference of the losses;
iterates and losses agree to 1e-3 relative as for the other drivers.
"""
import numpy as np
import pytest
import torch

import core_inputs
import oracle
from helpers import rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def core_mod():
    import paper_2309_13307_b200 as core_mod
    core_mod.lib()
    return core_mod


@pytest.mark.parametrize("n,rows,d,m,r1,H,c,iters,seed", [
    (3, 40, 512, 4, 0.1, 1.0, 1.0, 40, 6),            # second term of the rule decides
    (2, 64, 1001, 8, 0.02, 1e-4, 1.0, 30, 5),         # first term decides (constant step m / (16 r1))
    (20, 16, 300, 16, 0.05, 0.5, 2.0, 12, 3),         # more than one machine group
])
def test_option1_trajectory(core_mod, n, rows, d, m, r1, H, c, iters, seed):
    ls_in = core_inputs.least_squares(n=n, rows=rows, d=d, seed=11, decay=1.0, noise=0.05, device="cpu")
    A, b = ls_in.A.cuda(), ls_in.b.cuda()
    Ah, bh = ls_in.A.numpy(), ls_in.b.numpy()
    ctx = core_mod.Core(seed, d, m)
    ls = core_mod.LeastSquares(A, b)
    x = torch.zeros(d, dtype=torch.float32, device="cuda")
    f = ctx.core_ls_loss(ls, x).clone()
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    p_dev = torch.zeros(1, dtype=torch.float32, device="cuda")
    h_dev = torch.zeros(1, dtype=torch.float32, device="cuda")
    xo = np.zeros(d)
    fo = oracle.ls_loss(Ah, bh, xo)
    checked = 0
    for k in range(iters):
        xn, fn, acc, p, h = oracle.gd_step_option1(seed, k, m, Ah, bh, r1, H, c, xo, fo)
        trial = oracle.gd_step(seed, k, m, Ah, bh, h, xo)
        margin = abs(oracle.ls_loss(Ah, bh, trial) - fo)
        ctx.core_gd_step_option1(ls, r1, H, c, x, f, flag, p_dev, h_dev)
        assert ctx.core_get_round() == k + 1
        assert abs(p_dev.item() - p) <= 1e-4 * p, (k, p_dev.item(), p)
        assert abs(h_dev.item() - h) <= 1e-4 * h, (k, h_dev.item(), h)
        if margin <= 1e-4 * fo:
            break                                   # a near-tie: the two sides may part ways from here on
        assert bool(flag.item()) == acc, k
        xo, fo = xn, fn
        assert rel_l2(x.cpu().numpy(), xo) <= 1e-3 or float(np.abs(xo).max()) == 0.0, k
        assert abs(float(f.item()) - fo) <= 1e-3 * fo
        checked += 1
    assert checked >= min(iters, 8)
    assert core_mod.core_device_status() == 0


def test_option1_rejects_bad_constants_and_optional_outputs(core_mod):
    L = core_mod.lib()
    ls_in = core_inputs.least_squares(n=2, rows=30, d=260, seed=4, device="cuda")
    ctx = core_mod.Core(3, 260, 4)
    ls = core_mod.LeastSquares(ls_in.A, ls_in.b)
    x = torch.zeros(260, dtype=torch.float32, device="cuda")
    f = ctx.core_ls_loss(ls, x).clone()
    for r1, H, c in [(0.0, 1.0, 1.0), (1.0, -1.0, 1.0), (1.0, 1.0, 0.0), (float("nan"), 1.0, 1.0)]:
        assert L.core_gd_step_option1(ctx._h, ls._h, r1, H, c, x.data_ptr(), f.data_ptr(), None, None, None) == -1
    assert ctx.core_get_round() == 0
    f0 = f.clone()
    ctx.core_gd_step_option1(ls, 0.05, 1.0, 1.0, x, f)      # all optional outputs omitted
    torch.cuda.synchronize()
    assert ctx.core_get_round() == 1 and float(f.item()) <= float(f0.item())
