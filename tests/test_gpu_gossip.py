"""GPU parity of the decentralised variant (Algorithm 5: gossip averaging of the messages) against the oracle.

A gossip round is n multiply-adds per entry in fp32 with weights in [0, 1] that sum to one: compared with
the fp64 oracle to 1e-6 of the largest message.  The step's iterate follows the oracle's to 1e-3 relative
like the other drivers, its spread (how far from consensus the gossip stopped) to 1e-4 of the largest message.
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


@pytest.mark.parametrize("topology,n,m", [("ring", 8, 64), ("torus", 16, 130), ("complete", 5, 7), ("ring", 33, 1)])
def test_gossip_round_matches_oracle(core_mod, topology, n, m):
    W = core_inputs.gossip_matrix(topology, n)
    P = core_inputs.gradients(n, m, seed=3).numpy().astype(np.float64)
    ctx = core_mod.Core(1, 16, m)
    W_dev = torch.from_numpy(W.astype(np.float32)).cuda()
    cur = torch.from_numpy(P.astype(np.float32)).cuda()
    W32 = W.astype(np.float32).astype(np.float64)              # the weights the device actually holds
    scale = np.abs(P).max()
    for rounds in range(1, 6):
        cur = ctx.core_gossip_round(W_dev, cur)
        want = oracle.gossip_average(W32, P.astype(np.float32).astype(np.float64), rounds)
        assert np.abs(cur.cpu().numpy() - want).max() <= 1e-6 * scale, rounds
    L = core_mod.lib()
    assert L.core_gossip_round(ctx._h, W_dev.data_ptr(), cur.data_ptr(), n, cur.data_ptr()) == -1   # in place
    assert L.core_gossip_round(ctx._h, None, cur.data_ptr(), n, cur.data_ptr()) == -1


@pytest.mark.parametrize("topology,n,rounds,m", [("ring", 8, 6, 16), ("torus", 16, 10, 64), ("ring", 20, 3, 8)])
def test_decentralised_trajectory(core_mod, topology, n, rounds, m):
    d, rows, seed = 640, 24, 7
    ls_in = core_inputs.least_squares(n=n, rows=rows, d=d, seed=5, decay=1.0, noise=0.05, device="cpu")
    h = float(np.float32(0.5 / core_inputs.lipschitz_constant(ls_in.A, iters=60)))
    A, b = ls_in.A.cuda(), ls_in.b.cuda()
    Ah, bh = ls_in.A.numpy(), ls_in.b.numpy()
    W = core_inputs.gossip_matrix(topology, n)
    W_dev = torch.from_numpy(W.astype(np.float32)).cuda()
    W32 = W.astype(np.float32).astype(np.float64)
    ctx = core_mod.Core(seed, d, m)
    ls = core_mod.LeastSquares(A, b)
    x = torch.zeros(d, dtype=torch.float32, device="cuda")
    spread = torch.zeros(1, dtype=torch.float32, device="cuda")
    xo = np.zeros(d)
    reader = n // 3
    for k in range(15):
        G = oracle.ls_grad(Ah, bh, xo)
        biggest = float(np.abs(oracle.project(seed, k, m, G)).max())
        xo, spread_o = oracle.decentralized_step(seed, k, m, Ah, bh, W32, rounds, h, xo, reader=reader)
        ctx.core_decentralized_step(ls, W_dev, rounds, h, x, reader=reader, spread_dev=spread)
        assert ctx.core_get_round() == k + 1
        assert rel_l2(x.cpu().numpy(), xo) <= 1e-3, k
        assert abs(spread.item() - spread_o) <= 1e-4 * biggest, (k, spread.item(), spread_o)
    assert core_mod.core_device_status() == 0


def test_many_rounds_reach_the_centralised_step_and_printed_prefactor(core_mod):
    n, d, rows, m, seed = 8, 512, 32, 32, 2
    ls_in = core_inputs.least_squares(n=n, rows=rows, d=d, seed=9, decay=1.0, noise=0.05, device="cuda")
    h = float(np.float32(0.5 / core_inputs.lipschitz_constant(ls_in.A, iters=60)))
    W_dev = torch.from_numpy(core_inputs.gossip_matrix("complete", n).astype(np.float32)).cuda()
    ls = core_mod.LeastSquares(ls_in.A, ls_in.b)
    x0 = core_inputs.gradients(1, d, seed=4, device="cuda")[0].contiguous()
    central, gossip, printed = x0.clone(), x0.clone(), x0.clone()
    core_mod.Core(seed, d, m).core_gd_step(ls, h, central)
    spread = torch.ones(1, dtype=torch.float32, device="cuda")
    core_mod.Core(seed, d, m).core_decentralized_step(ls, W_dev, 2, h, gossip, reader=5, spread_dev=spread)
    core_mod.Core(seed, d, m).core_decentralized_step(ls, W_dev, 2, h / n, printed, reader=0, as_printed=True)
    step = float(torch.linalg.vector_norm(central - x0))
    assert float(torch.linalg.vector_norm(gossip - central)) <= 1e-4 * step
    assert float(torch.linalg.vector_norm(printed - central)) <= 1e-4 * step
    assert spread.item() <= 1e-5 * float(central.abs().max() + 1)
    # bad arguments are refused before anything is launched
    L = core_mod.lib()
    ctx = core_mod.Core(seed, d, m)
    assert L.core_decentralized_step(ctx._h, ls._h, W_dev.data_ptr(), 2, n, 0, h, x0.data_ptr(), None) == -1
    assert L.core_decentralized_step(ctx._h, ls._h, W_dev.data_ptr(), -1, 0, 0, h, x0.data_ptr(), None) == -1
    assert L.core_decentralized_step(ctx._h, ls._h, None, 2, 0, 0, h, x0.data_ptr(), None) == -1
    assert ctx.core_get_round() == 0
