"""The machine-per-rank harness with the CUDA library as its engine, one rank over NCCL on one GPU.

With a single rank the exchange is trivial, but every call of the harness goes through the C ABI and the
collective runs over NCCL on device buffers; the result must be the oracle's round for one machine.  (More
ranks need more GPUs; the exchange itself is covered on CPU ranks in test_machine_per_rank.py.)
"""
import socket

import numpy as np
import pytest
import torch

import core_inputs
import oracle
from helpers import P_TOL, REC_TOL, rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture()
def one_rank_group():
    import torch.distributed as dist
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                            device_id=torch.device("cuda", 0))
    yield dist
    dist.destroy_process_group()


def test_one_machine_round_matches_the_oracle(one_rank_group):
    import paper_2309_13307_b200 as core_mod
    from paper_2309_13307_b200.machine_per_gpu import MachinePerRank
    seed, d, m = 4, 100_003, 48
    G = core_inputs.gradients(1, d, seed=8, device="cuda")
    ctx = core_mod.Core(seed, d, m)
    ctx.core_set_round(2)
    machine = MachinePerRank(ctx, m)
    pbar, gt = machine.core_round(G[0])
    W = torch.ones((1, 1), dtype=torch.float32, device="cuda")
    est, gt_dec = machine.core_round_decentralized(G[0], W, 2)
    torch.cuda.synchronize()
    assert ctx.core_get_round() == 4 and core_mod.core_device_status() == 0
    Gh = core_inputs.to_oracle_array(G)
    norm = float(np.sqrt((Gh.astype(np.float64) ** 2).sum()))
    _, pbar_o, gt_o = oracle.core_round(seed, 2, m, Gh)
    assert np.abs(pbar.cpu().numpy() - pbar_o).max() <= P_TOL * norm
    assert rel_l2(gt.cpu().numpy(), gt_o) <= REC_TOL
    _, est_o, gt_dec_o = oracle.core_round(seed, 3, m, Gh)           # one machine: gossip leaves it alone
    assert np.abs(est.cpu().numpy() - est_o).max() <= P_TOL * norm
    assert rel_l2(gt_dec.cpu().numpy(), gt_dec_o) <= REC_TOL
    ctx.close()
