"""Error behaviour of the C ABI on a live device: bad arguments return CORE_EINVAL and launch nothing;
contexts keep working afterwards.  (No test here faults the GPU: every rejected call returns on the host.)"""
import ctypes

import pytest
import torch

import core_inputs

pytestmark = pytest.mark.gpu

EINVAL = -1


@pytest.fixture(scope="module")
def core_mod():
    import paper_2309_13307_b200 as core_mod
    core_mod.lib()
    return core_mod


def test_round_entry_points_reject_bad_arguments(core_mod):
    L = core_mod.lib()
    d, m, n = 1000, 8, 2
    ctx = core_mod.Core(1, d, m)
    G = core_inputs.gradients(n, d, seed=1, device="cuda")
    P = torch.full((n, m), 7.0, dtype=torch.float32, device="cuda")
    pbar = torch.full((m,), 7.0, dtype=torch.float32, device="cuda")
    gt = torch.full((d,), 7.0, dtype=torch.float32, device="cuda")
    h = ctx._h
    assert L.core_project(h, None, 0, n, d, P.data_ptr()) == EINVAL
    assert L.core_project(h, G.data_ptr(), 0, n, d, None) == EINVAL
    assert L.core_project(h, G.data_ptr(), 0, 0, d, P.data_ptr()) == EINVAL            # n < 1
    assert L.core_project(h, G.data_ptr(), 0, n, d - 1, P.data_ptr()) == EINVAL        # ld < d
    assert L.core_project(h, G.data_ptr(), 5, n, d, P.data_ptr()) == EINVAL            # unknown dtype
    assert L.core_project(None, G.data_ptr(), 0, n, d, P.data_ptr()) == EINVAL
    assert L.core_aggregate(h, None, n, pbar.data_ptr()) == EINVAL
    assert L.core_aggregate(h, P.data_ptr(), 0, pbar.data_ptr()) == EINVAL
    assert L.core_reconstruct(h, None, gt.data_ptr()) == EINVAL
    assert L.core_reconstruct(h, pbar.data_ptr(), None) == EINVAL
    assert L.core_round(h, G.data_ptr(), 0, n, d, None, gt.data_ptr()) == EINVAL
    assert L.core_round_host(h, None, 0, n, d, None, None) == EINVAL
    assert L.core_debug_philox(h, 0, 0, 4, ctypes.c_void_p(P.data_ptr() + 4)) == EINVAL   # misaligned window
    torch.cuda.synchronize()
    # nothing was written by the rejected calls, the round counter did not move
    assert float(P.min()) == 7.0 and float(pbar.min()) == 7.0 and float(gt.min()) == 7.0
    assert ctx.core_get_round() == 0
    # and the context still works
    ctx.core_project(G, P)
    torch.cuda.synchronize()
    assert float(P.abs().max()) != 7.0
    assert L.core_strerror(-4) == b"size exceeds the fixed capacity of this entry point"


def test_least_squares_entry_points_reject_bad_arguments(core_mod):
    L = core_mod.lib()
    ls_in = core_inputs.least_squares(n=2, rows=8, d=64, seed=1, device="cuda")
    ls = core_mod.LeastSquares(ls_in.A, ls_in.b)
    ctx_ok = core_mod.Core(1, 64, 4)
    ctx_other_d = core_mod.Core(1, 128, 4)
    x = torch.zeros(64, dtype=torch.float32, device="cuda")
    x128 = torch.zeros(128, dtype=torch.float32, device="cuda")
    hdl = ctypes.c_void_p()
    assert L.core_ls_create(ctypes.byref(hdl), None, ls_in.b.data_ptr(), 2, 8, 64) == EINVAL
    assert L.core_ls_create(ctypes.byref(hdl), ls_in.A.data_ptr(), ls_in.b.data_ptr(), 2, 0, 64) == EINVAL
    assert hdl.value is None
    assert L.core_gd_step(ctx_other_d._h, ls._h, 0.1, x128.data_ptr()) == EINVAL          # d mismatch
    assert L.core_gd_step(ctx_ok._h, None, 0.1, x.data_ptr()) == EINVAL
    assert L.core_agd_step(ctx_ok._h, ls._h, 0.1, 0.5, x.data_ptr(), x.data_ptr()) == EINVAL   # x and x_prev alias
    assert L.core_gd_step_guarded(ctx_ok._h, ls._h, 0.1, x.data_ptr(), None, None) == EINVAL
    assert ctx_ok.core_get_round() == 0
    ctx_ok.core_gd_step(ls, 0.1, x)
    torch.cuda.synchronize()
    assert ctx_ok.core_get_round() == 1 and bool(torch.isfinite(x).all())
