"""core_project_static: the projection for callers that are not allowed to allocate.

Some users of this library run where cudaMalloc is off limits: their memory pool owns the
whole device, or they sit on a path that must not trigger the allocator's device-wide
synchronisation.  For them the library has one entry point that needs no context and no
workspace: its scratch is a fixed 4 MiB array inside the library.  This file checks, through
the C ABI, that it returns what core_project returns (same tolerance as the other parity
tests: |dP| <= 1e-4 ||g_i||), on two calls in a row that share the array, that device memory
does not move across the calls, and that sizes beyond the array are refused.

The file name makes pytest collect it last, so a failure here cannot hide the other tests
from a run that stops at the first failure; it also passes when run alone.
"""
import ctypes

import numpy as np
import pytest
import torch

import core_inputs
from helpers import P_TOL

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def core_mod():
    import paper_2309_13307_b200 as core_mod
    core_mod.lib()
    return core_mod


def reference_projection(core_mod, seed, t, m, G):
    ctx = core_mod.Core(seed, G.shape[1], m)
    ctx.core_set_round(t)
    P = ctx.core_project(G)
    torch.cuda.synchronize()
    ctx.close()
    return P


def test_two_calls_in_a_row_match_core_project(core_mod):
    cases = [
        # (seed, t, n, m, d, dtype): the second call is larger than the first and leaves no
        # room for stale partial sums of the first to go unnoticed; the third fills a quarter of the
        # array; the fourth needs more CTA columns than fit (see the check below) and runs with fewer
        (1, 0, 4, 16, 4096, "f32"),
        (7, 3, 2, 64, 1_000_003, "f32"),
        (9, 1, 16, 1024, 300_000, "bf16"),
        (5, 2, 8, 512, 1_000_003, "f32"),
    ]
    # the fourth case really is clamped: its usual plan wants more partial sums than the array holds
    from paper_2309_13307_b200 import binding
    sm_count = torch.cuda.get_device_properties(0).multi_processor_count
    plan = binding.core_debug_project_plan(8, 512, 1_000_003, binding.CORE_F32, sm_count)
    assert plan["grid_x"] * 8 * 512 > binding.CORE_STATIC_SCRATCH_FLOATS
    inputs = [core_inputs.gradients(n, d, seed=10 + k, dtype=dt, device="cuda")
              for k, (_, _, n, m, d, dt) in enumerate(cases)]
    want = [reference_projection(core_mod, s, t, m, G) for (s, t, n, m, d, dt), G in zip(cases, inputs)]
    outs = [torch.full((n, m), float("nan"), dtype=torch.float32, device="cuda") for (_, _, n, m, _, _) in cases]
    # the first call on the device looks up the array's address; do it before measuring memory
    core_mod.core_project_static(cases[0][0], cases[0][1], cases[0][3], inputs[0], outs[0])
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for rep in range(2):                                   # back to back, sharing the array
        for (s, t, n, m, d, dt), G, out in zip(cases, inputs, outs):
            out.fill_(float("nan"))
            core_mod.core_project_static(s, t, m, G, out)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before                       # nothing was allocated or freed
    for (s, t, n, m, d, dt), G, out, ref in zip(cases, inputs, outs, want):
        norms = torch.linalg.vector_norm(G.float(), dim=1).double().cpu().numpy()
        diff = np.abs(out.cpu().numpy().astype(np.float64) - ref.cpu().numpy().astype(np.float64))
        assert np.isfinite(out.cpu().numpy()).all()
        assert (diff <= P_TOL * norms[:, None]).all(), float((diff / norms[:, None]).max())
    # same launch geometry as core_project: bitwise the same
    assert torch.equal(outs[0], want[0]) and torch.equal(outs[1], want[1])
    # and against the oracle directly (one machine, two vectors of the clamped case)
    import oracle
    from helpers import oracle_project_entry
    s, t, n, m, d, dt = cases[3]
    row = core_inputs.to_oracle_array(inputs[3][2:3])[0]
    norm = float(np.sqrt((row.astype(np.float64) ** 2).sum()))
    for j in (0, m - 1):
        assert abs(float(outs[3][2, j]) - oracle_project_entry(s, t, j, row)) <= P_TOL * norm


def test_first_call_on_a_device_is_the_set_up_call(core_mod):
    """What the header documents: later calls leave free device memory untouched; the first call in a
    process may load the library's code and its 4 MiB array (lazy module loading), so its own delta is
    recorded rather than required to be zero."""
    G = core_inputs.gradients(2, 4096, seed=3, device="cuda")
    P = torch.empty((2, 8), dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    core_mod.core_project_static(1, 0, 8, G, P)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    core_mod.core_project_static(1, 0, 8, G, P)
    torch.cuda.synchronize()
    free2, _ = torch.cuda.mem_get_info()
    print(f"first call moved free memory by {free0 - free1} bytes, second by {free1 - free2}")
    assert free2 == free1
    assert 0 <= free0 - free1 <= 64 << 20


def test_buffers_of_another_kind_are_refused(core_mod):
    L = core_mod.lib()
    G = core_inputs.gradients(2, 64, seed=1, device="cuda")
    P_host = torch.zeros((2, 4), dtype=torch.float32).pin_memory()
    err = ctypes.c_int(0)
    rc = L.core_project_static(1, 0, 64, 4, G.data_ptr(), 0, 2, 64, P_host.data_ptr(), None, ctypes.byref(err))
    assert rc == -1                                           # a host pointer is not this device's memory


def test_sizes_beyond_the_array_are_refused(core_mod):
    G = core_inputs.gradients(17, 64, seed=1, device="cuda")
    P = torch.zeros((17, 4), dtype=torch.float32, device="cuda")
    with pytest.raises(core_mod.CoreError) as err:
        core_mod.core_project_static(1, 0, 4, G, P)        # more than 16 machines
    assert err.value.code == core_mod.CORE_ELIMIT
    m = (1 << 20) // 2 + 1                                  # n * m just over 2^20 floats
    G = core_inputs.gradients(2, 64, seed=1, device="cuda")
    P = torch.zeros((2, m), dtype=torch.float32, device="cuda")
    with pytest.raises(core_mod.CoreError) as err:
        core_mod.core_project_static(1, 0, m, G, P)
    assert err.value.code == core_mod.CORE_ELIMIT
    assert float(P.abs().max()) == 0.0                      # nothing was launched
    # exactly at the limit is accepted
    m = (1 << 20) // 2
    P = torch.zeros((2, m), dtype=torch.float32, device="cuda")
    core_mod.core_project_static(1, 0, m, G, P)
    torch.cuda.synchronize()
    assert bool(torch.isfinite(P).all()) and float(P.abs().max()) > 0.0
