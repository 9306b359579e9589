"""Failure paths on a live device, made without faulting, trapping or hanging the GPU.

* Out of memory is injected on the host (core_debug_fail_allocations): the entry points return
  CORE_ENOMEM, launch nothing, and their contexts keep working.
* A bounded device-side wait is made to run out by waiting on a barrier that nobody completes (a small
  test kernel that uses the projection's own wait helper): the kernel returns by its normal exit, the
  status word carries the code, and the device keeps working.
"""
import ctypes

import numpy as np
import pytest
import torch

import core_inputs

pytestmark = pytest.mark.gpu

ENOMEM = -2


@pytest.fixture(scope="module")
def core_mod():
    import paper_2309_13307_b200 as core_mod
    core_mod.lib()
    return core_mod


@pytest.fixture()
def binding(core_mod):
    from paper_2309_13307_b200 import binding
    yield binding
    binding.core_debug_fail_allocations(0)            # never leave the hook armed for other tests


def test_core_init_reports_out_of_memory(core_mod, binding):
    L = core_mod.lib()
    binding.core_debug_fail_allocations(1)
    h = ctypes.c_void_p()
    assert L.core_init(ctypes.byref(h), 1, 4096, 16) == ENOMEM
    assert h.value is None
    # the hook is spent: the next context is created normally
    ctx = core_mod.Core(1, 4096, 16)
    assert ctx.core_workspace_bytes() == 16 * 4


def test_project_and_reserve_report_out_of_memory_and_recover(core_mod, binding):
    L = core_mod.lib()
    n, d, m = 4, 100_000, 16
    G = core_inputs.gradients(n, d, seed=1, device="cuda")
    ctx = core_mod.Core(1, d, m)
    P = torch.full((n, m), 7.0, dtype=torch.float32, device="cuda")
    binding.core_debug_fail_allocations(1)
    assert L.core_project(ctx._h, G.data_ptr(), 0, n, d, P.data_ptr()) == ENOMEM
    torch.cuda.synchronize()
    assert float(P.min()) == 7.0 and float(P.max()) == 7.0            # nothing was launched
    assert L.core_last_cuda_error(ctx._h) == 2                         # cudaErrorMemoryAllocation
    binding.core_debug_fail_allocations(1)
    assert L.core_reserve_workspace(ctx._h, n, 0) == ENOMEM
    assert ctx.core_workspace_bytes() == m * 4                         # no workspace yet
    # recovery: reserve, then project without a further allocation (the armed hook is not consumed)
    ctx.core_reserve_workspace(n)
    held = ctx.core_workspace_bytes()
    assert held > m * 4
    binding.core_debug_fail_allocations(1)
    ctx.core_project(G, P)
    pbar, gt = ctx.core_round(G)
    torch.cuda.synchronize()
    assert ctx.core_workspace_bytes() == held
    binding.core_debug_fail_allocations(0)
    want = core_mod.Core(1, d, m).core_project(G)
    assert torch.equal(P, want)
    assert L.core_reserve_workspace(ctx._h, 0, 0) == -1 and L.core_reserve_workspace(ctx._h, n, 9) == -1


def test_round_host_reports_out_of_memory_and_recovers(core_mod, binding):
    L = core_mod.lib()
    n, d, m = 2, 50_000, 8
    Gh = core_inputs.gradients(n, d, seed=2).pin_memory()
    pbar_h = torch.full((m,), 7.0, dtype=torch.float32).pin_memory()
    gt_h = torch.full((d,), 7.0, dtype=torch.float32).pin_memory()
    ctx = core_mod.Core(3, d, m)
    for fail in (1, 2):                        # the slabs, then (slabs granted) the workspace
        binding.core_debug_fail_allocations(fail)
        rc = L.core_round_host(ctx._h, Gh.data_ptr(), 0, n, d, pbar_h.data_ptr(), gt_h.data_ptr())
        binding.core_debug_fail_allocations(0)
        if rc == 0:
            break
        assert rc == ENOMEM
        assert float(gt_h.min()) == 7.0 and float(pbar_h.min()) == 7.0 and ctx.core_get_round() == 0
    ctx.core_set_round(0)
    ctx.core_round_host(Gh, pbar_h, gt_h)
    dev = core_mod.Core(3, d, m)
    pbar_d, gt_d = dev.core_round(Gh.cuda())
    torch.cuda.synchronize()
    assert np.allclose(gt_h.numpy(), gt_d.cpu().numpy(), rtol=0, atol=1e-5 * float(gt_d.abs().max()))


def test_least_squares_handle_reports_out_of_memory(core_mod, binding):
    L = core_mod.lib()
    ls_in = core_inputs.least_squares(n=2, rows=8, d=64, seed=1, device="cuda")
    binding.core_debug_fail_allocations(1)
    h = ctypes.c_void_p()
    assert L.core_ls_create(ctypes.byref(h), ls_in.A.data_ptr(), ls_in.b.data_ptr(), 2, 8, 64) == ENOMEM
    assert h.value is None
    core_mod.LeastSquares(ls_in.A, ls_in.b)


def test_a_bounded_wait_that_runs_out_is_reported_and_the_device_survives(core_mod, binding):
    assert core_mod.core_device_status() == 0
    served, seen = binding.core_debug_wait_timeout(200, 7)            # 200 microseconds
    assert served == 0 and seen == 1
    assert core_mod.core_device_status() == 7                         # the code, once
    assert core_mod.core_device_status() == 0
    # two in a row keep the larger code
    binding.core_debug_wait_timeout(50, 3)
    binding.core_debug_wait_timeout(50, 9)
    assert core_mod.core_device_status() == 9
    L = core_mod.lib()
    out = (ctypes.c_uint32 * 2)()
    assert L.core_debug_wait_timeout(0, 1, out) == -1 and L.core_debug_wait_timeout(10, 0, out) == -1
    assert L.core_debug_wait_timeout(10, 1, None) == -1
    # the device still computes, tensor-memory projection included
    G = core_inputs.gradients(16, 40_001, seed=5, dtype="bf16", device="cuda")
    ctx = core_mod.Core(2, 40_001, 256)
    a = ctx.core_project(G)
    b = ctx.core_project(G)
    assert torch.equal(a, b) and bool(torch.isfinite(a).all())
    assert core_mod.core_device_status() == 0


def test_loss_to_host_and_reserve(core_mod):
    ls_in = core_inputs.least_squares(n=3, rows=40, d=256, seed=4, device="cuda")
    ls = core_mod.LeastSquares(ls_in.A, ls_in.b)
    ctx = core_mod.Core(1, 256, 8)
    x = torch.randn(256, device="cuda")
    loss_h = torch.zeros(1, dtype=torch.float64).pin_memory()
    ctx.core_ls_loss_host(ls, x, loss_h)
    loss_d = ctx.core_ls_loss(ls, x)
    torch.cuda.synchronize()
    assert float(loss_h[0]) == float(loss_d[0]) and float(loss_h[0]) > 0
