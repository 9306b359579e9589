"""One machine of the paper per rank: the deployment Algorithm 2 describes.

Algorithm 2: machine i holds its own gradient g_i, sends the m numbers p_ij = <g_i, xi_j> to the
central machine, which returns their combination, and every machine reconstructs the same estimate
from it with the common vectors.  Here a rank is a machine (one process per GPU): the projection of the
local gradient and the reconstruction run in the library's kernels on the rank's GPU, and the exchange
is one collective of m floats per rank over ``torch.distributed`` (NCCL on GPUs).  The messages are
gathered, not summed in flight, and combined by ``core_aggregate`` in ascending machine order, so every
rank holds bitwise the same mean, and the same one the single-GPU simulation of n machines produces.

Algorithm 5 (decentralised): no central machine.  In a gossip round every rank sends its current
estimate of the mean message to its neighbours in the network W (the machines l with W[i][l] != 0) and
replaces it by sum_l W[i][l] estimate_l, l ascending, through ``core_gossip_round`` on a buffer whose
other rows are zero (a zero weight times a zero row adds nothing, so the result is row i of the full
product, bit for bit).

This file holds no arithmetic of the method: it moves m floats between ranks and calls the engine.
The engine is the CUDA binding's ``Core`` (there is no CPU implementation behind it); tests on CPU ranks
pass a stand-in with the same five methods.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


class MachinePerRank:
    """Rank r of the group plays machine r.

    engine: object with core_project(G[1 x d]) -> P[1 x m], core_aggregate(P[n x m]) -> pbar[m],
            core_reconstruct(pbar) -> gtilde[d], core_gossip_round(W, P_in, P_out) -> P_out,
            core_get_round() / core_set_round(t); all ranks' engines share (seed, d, m) and the round.
    """

    def __init__(self, engine, m: int, group=None):
        if not dist.is_initialized():
            raise RuntimeError("torch.distributed is not initialised: one process per machine is required")
        self.engine = engine
        self.m = int(m)
        self.group = group
        self.rank = dist.get_rank(group)
        self.n = dist.get_world_size(group)

    # ---- Algorithm 2: through a central combination ------------------------------------------
    def core_round(self, g_local: torch.Tensor):
        """One round: returns (pbar, gtilde), the same on every rank, and advances the round."""
        P_own = self.engine.core_project(g_local.reshape(1, -1))
        P_all = torch.empty((self.n, self.m), dtype=P_own.dtype, device=P_own.device)
        dist.all_gather_into_tensor(P_all, P_own.reshape(1, self.m).contiguous(), group=self.group)
        pbar = self.engine.core_aggregate(P_all)
        gtilde = self.engine.core_reconstruct(pbar)
        self.engine.core_set_round(self.engine.core_get_round() + 1)
        return pbar, gtilde

    # ---- Algorithm 5: gossip with the neighbours only ----------------------------------------
    def neighbours(self, W: torch.Tensor):
        row = W[self.rank].detach().cpu()
        return [l for l in range(self.n) if l != self.rank and float(row[l]) != 0.0]

    def gossip_round(self, W: torch.Tensor, estimate: torch.Tensor) -> torch.Tensor:
        """estimate (m floats, this machine's) -> sum_l W[rank][l] estimate_l after one exchange."""
        near = self.neighbours(W)
        P_in = torch.zeros((self.n, self.m), dtype=estimate.dtype, device=estimate.device)
        P_in[self.rank].copy_(estimate)
        if near:
            ops = []
            for l in near:
                ops.append(dist.P2POp(dist.isend, estimate, l, group=self.group))
                ops.append(dist.P2POp(dist.irecv, P_in[l], l, group=self.group))
            for req in dist.batch_isend_irecv(ops):
                req.wait()
        P_out = torch.empty_like(P_in)
        self.engine.core_gossip_round(W, P_in, P_out)
        return P_out[self.rank].clone()

    def core_round_decentralized(self, g_local: torch.Tensor, W: torch.Tensor, rounds: int):
        """Projection, `rounds` gossip rounds, reconstruction from this machine's own estimate.

        Returns (estimate, gtilde): they differ between ranks by what the gossip has left of the
        disagreement; the round advances on every rank."""
        estimate = self.engine.core_project(g_local.reshape(1, -1)).reshape(self.m)
        for _ in range(int(rounds)):
            estimate = self.gossip_round(W, estimate)
        gtilde = self.engine.core_reconstruct(estimate)
        self.engine.core_set_round(self.engine.core_get_round() + 1)
        return estimate, gtilde
