"""The machine-per-rank deployment (Algorithm 2's exchange; Algorithm 5's gossip) on CPU ranks over gloo.

The harness under test moves m floats between ranks and calls its engine; on a GPU the engine is the
CUDA library, here it is a stand-in that answers from the oracle, so what is checked is the exchange:
that the combined message and the estimate on every rank are the oracle's for the stacked gradients, and
that rank i's gossip estimate after K rounds is row i of the oracle's W^K P.
"""
import os
import pickle
import socket
import sys

import numpy as np
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SEED, D, M = 5, 256, 12


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


class OracleEngine:
    """The five calls the harness makes, answered by the oracle in fp64 (CPU tensors in and out)."""

    def __init__(self, seed, d, m):
        import oracle
        self.o, self.seed, self.d, self.m, self.t = oracle, seed, d, m, 0

    def core_get_round(self):
        return self.t

    def core_set_round(self, t):
        self.t = t

    def core_project(self, G):
        return torch.from_numpy(self.o.project(self.seed, self.t, self.m, G.numpy().astype(np.float32)))

    def core_aggregate(self, P):
        return torch.from_numpy(self.o.aggregate(P.numpy()))

    def core_reconstruct(self, pbar):
        return torch.from_numpy(self.o.reconstruct(self.seed, self.t, pbar.numpy(), self.d))

    def core_gossip_round(self, W, P_in, P_out):
        P_out.copy_(torch.from_numpy(self.o.gossip_round(W.numpy(), P_in.numpy())))
        return P_out


def gradients(n):
    import core_inputs
    return core_inputs.gradients(n, D, seed=3, device="cpu")


def worker(rank, world, port, topology, rounds, out_dir):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import core_inputs
    from paper_2309_13307_b200.machine_per_gpu import MachinePerRank
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    G = gradients(world)
    machine = MachinePerRank(OracleEngine(SEED, D, M), M)
    pbar, gt = machine.core_round(G[rank])
    W = torch.from_numpy(core_inputs.gossip_matrix(topology, world))
    est, gt_dec = machine.core_round_decentralized(G[rank], W, rounds)
    with open(os.path.join(out_dir, f"r{rank}.pkl"), "wb") as f:
        pickle.dump({"pbar": pbar.numpy(), "gt": gt.numpy(), "est": est.numpy(), "gt_dec": gt_dec.numpy(),
                     "t": machine.engine.core_get_round(), "near": machine.neighbours(W)}, f)
    dist.barrier()
    dist.destroy_process_group()


def run(world, topology, rounds, tmp_path):
    mp.spawn(worker, args=(world, free_port(), topology, rounds, str(tmp_path)), nprocs=world, join=True)
    return [pickle.load(open(tmp_path / f"r{r}.pkl", "rb")) for r in range(world)]


def test_two_machines_agree_with_the_oracle_round(tmp_path):
    import oracle
    world = 2
    got = run(world, "ring", 3, tmp_path)
    G = gradients(world).numpy()
    P, pbar, gt = oracle.core_round(SEED, 0, M, G)
    for r in range(world):
        assert np.array_equal(got[r]["pbar"], pbar)            # same numbers in the same order
        assert np.array_equal(got[r]["gt"], gt)
        assert got[r]["t"] == 2                                # two rounds were played
    # the second round (t = 1) was the decentralised one
    P1 = oracle.project(SEED, 1, M, G)
    W = __import__("core_inputs").gossip_matrix("ring", world)
    want = oracle.gossip_average(W, P1, 3)
    for r in range(world):
        assert np.allclose(got[r]["est"], want[r], rtol=0, atol=1e-12 * np.abs(P1).max())
        assert np.array_equal(got[r]["gt_dec"], oracle.reconstruct(SEED, 1, got[r]["est"], D))


def test_four_machines_on_a_ring_talk_to_their_neighbours_only(tmp_path):
    import core_inputs
    import oracle
    world, rounds = 4, 5
    got = run(world, "ring", rounds, tmp_path)
    G = gradients(world).numpy()
    W = core_inputs.gossip_matrix("ring", world)
    P1 = oracle.project(SEED, 1, M, G)
    want = oracle.gossip_average(W, P1, rounds)
    mean = P1.mean(axis=0)
    for r in range(world):
        assert got[r]["near"] == sorted({(r - 1) % world, (r + 1) % world})
        assert np.allclose(got[r]["est"], want[r], rtol=0, atol=1e-12 * np.abs(P1).max())
    # the estimates contract towards the mean message at the rate of W's second eigenvalue (1/3 here)
    before = np.abs(P1 - mean).max()
    after = max(np.abs(got[r]["est"] - mean).max() for r in range(world))
    assert after <= before * (1.0 / 3.0) ** rounds * 4.0
