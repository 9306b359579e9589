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
        # room for stale partial sums of the first to go unnoticed; the third forces fewer CTA
        # columns than core_project uses (16 * 1024 floats per column, 64 columns fit)
        (1, 0, 4, 16, 4096, "f32"),
        (7, 3, 2, 64, 1_000_003, "f32"),
        (9, 1, 16, 1024, 300_000, "bf16"),
    ]
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
