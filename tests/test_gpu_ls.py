"""GPU parity of the machine gradients g_i = A_i^T (A_i x - b_i) / rows of the least-squares driver
(Algorithm 2's local computation) for both device paths: the single pass over A (d <= 8192, d % 4 == 0,
16-byte aligned x) and the two-pass path (any shape).  Bar: relative L2 <= 1e-5 per machine against the
fp64 oracle."""
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


@pytest.mark.parametrize("n,rows,d", [(1, 1, 4), (2, 7, 1024), (3, 50, 1028), (8, 300, 8192), (4, 33, 2052),
                                      (2, 5, 8196), (3, 20, 1001), (40, 9, 512)])
def test_gradients_both_paths(core_mod, n, rows, d):
    ls_in = core_inputs.least_squares(n=n, rows=rows, d=d, seed=n + rows, device="cuda")
    ls = core_mod.LeastSquares(ls_in.A, ls_in.b)
    ctx = core_mod.Core(1, d, 4)
    store = core_inputs.gradients(1, d + 4, seed=3, device="cuda")[0].contiguous()
    x_aligned = store[:d].clone()
    x_shifted = store[1:d + 1]                      # 4-byte offset: forces the two-pass path
    Ah, bh = ls_in.A.cpu().numpy(), ls_in.b.cpu().numpy()
    for x in (x_aligned, x_shifted):
        G = ctx.core_ls_gradients(ls, x.contiguous() if x is x_aligned else x).cpu().numpy()
        Go = oracle.ls_grad(Ah, bh, x.cpu().numpy().astype(np.float64))
        for i in range(n):
            assert rel_l2(G[i], Go[i]) <= 1e-5, (i, rel_l2(G[i], Go[i]))
    # both paths at the same point agree closely and each is bitwise reproducible
    xs = x_aligned.clone()
    a = ctx.core_ls_gradients(ls, xs)
    b = ctx.core_ls_gradients(ls, xs)
    assert torch.equal(a, b)
