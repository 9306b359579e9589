"""Run state and memory hygiene of the CUDA path.

* Resume: the whole state of a run is (seed, round index t, x, x_prev), because the common vectors are a
  pure function of (seed, t, j, coordinate).  A run interrupted and resumed from that state in a fresh
  context must continue bit for bit.
* Canaries: no entry point writes outside the extents its contract states (sentinel words around every
  output are checked after the calls).
"""
import pytest
import torch

import core_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def core_mod():
    import paper_2309_13307_b200 as core_mod
    core_mod.lib()
    return core_mod


def test_resume_from_seed_round_and_iterates_is_bitwise(core_mod):
    ls_in = core_inputs.least_squares(n=3, rows=40, d=2052, seed=1, device="cuda")
    d, m, h, beta = 2052, 8, 0.2, 0.3
    ls = core_mod.LeastSquares(ls_in.A, ls_in.b)

    def fresh():
        return (torch.zeros(d, dtype=torch.float32, device="cuda"), torch.zeros(d, dtype=torch.float32, device="cuda"))

    ctx = core_mod.Core(77, d, m)
    x, xp = fresh()
    for _ in range(3):
        ctx.core_gd_step(ls, h, x)
    for _ in range(4):
        ctx.core_agd_step(ls, h, beta, x, xp)
    straight = (x.clone(), xp.clone(), ctx.core_get_round())

    ctx1 = core_mod.Core(77, d, m)
    x, xp = fresh()
    for _ in range(3):
        ctx1.core_gd_step(ls, h, x)
    for _ in range(2):
        ctx1.core_agd_step(ls, h, beta, x, xp)
    saved = (x.clone(), xp.clone(), ctx1.core_get_round())
    ctx1.close()

    ctx2 = core_mod.Core(77, d, m)                      # a new context, as after a restart
    ctx2.core_set_round(saved[2])
    x, xp = saved[0].clone(), saved[1].clone()
    for _ in range(2):
        ctx2.core_agd_step(ls, h, beta, x, xp)
    assert ctx2.core_get_round() == straight[2] == 7
    assert torch.equal(x, straight[0]) and torch.equal(xp, straight[1])


def guarded(numel, dtype=torch.float32, pad=64, fill=-12345.0):
    """A view of `numel` elements with `pad` sentinel elements on both sides (16-byte aligned start)."""
    store = torch.full((numel + 2 * pad,), fill, dtype=dtype, device="cuda")
    return store, store[pad:pad + numel]


def sentinels_intact(store, numel, pad=64, fill=-12345.0):
    return bool((store[:pad] == fill).all()) and bool((store[pad + numel:] == fill).all())


@pytest.mark.parametrize("n,m,d,dtype", [(4, 16, 4096, "f32"), (3, 7, 5003, "bf16"), (17, 5, 1001, "f32")])
def test_no_writes_outside_the_outputs(core_mod, n, m, d, dtype):
    G = core_inputs.gradients(n, d, seed=3, dtype=dtype, device="cuda")
    ctx = core_mod.Core(5, d, m)
    Ps, P = guarded(n * m)
    ps, pbar = guarded(m)
    gs, gt = guarded(d)
    ctx.core_project(G, P.view(n, m))
    ctx.core_aggregate(P.view(n, m), pbar)
    ctx.core_reconstruct(pbar, gt)
    ctx.core_round(G, pbar, gt)
    core_mod.core_project_static(5, 0, m, G[:min(n, 16)], P[:min(n, 16) * m].view(min(n, 16), m))
    torch.cuda.synchronize()
    assert sentinels_intact(Ps, n * m) and sentinels_intact(ps, m) and sentinels_intact(gs, d)
    assert bool(torch.isfinite(gt).all()) and bool(torch.isfinite(P).all())
    # least-squares steps: x and x_prev
    ls_in = core_inputs.least_squares(n=2, rows=16, d=d, seed=2, device="cuda")
    ls = core_mod.LeastSquares(ls_in.A, ls_in.b)
    xs, x = guarded(d, fill=0.0)
    xs[:64] = -12345.0
    xs[64 + d:] = -12345.0
    xps, xp = guarded(d, fill=0.0)
    xps[:64] = -12345.0
    xps[64 + d:] = -12345.0
    ctx.core_gd_step(ls, 0.1, x)
    ctx.core_agd_step(ls, 0.1, 0.5, x, xp)
    f = ctx.core_ls_loss(ls, x).clone()
    ctx.core_gd_step_guarded(ls, 0.1, x, f)
    torch.cuda.synchronize()
    assert sentinels_intact(xs, d) and sentinels_intact(xps, d)
