"""Seeded synthetic inputs for the CORE round.

This module only manufactures inputs (gradients, least-squares problems); it
holds none of the method's arithmetic.  Both the CUDA tests/benchmark and the
CPU oracle consume the arrays made here, so the two sides always see
bit-identical numbers: bf16 inputs are rounded once, here, before either side
looks at them.

Every generator takes a ``device``; values are drawn with a ``torch.Generator``
seeded from ``seed`` on that device.  (The CPU and CUDA generators produce
different streams; a test always hands one and the same array to both sides.)

Workloads (shapes and distributions of the evaluation configurations):
  tiny        d=4096       n=4   m=16    fp32  N(0,1)
  resnet50    d=25,557,032 n=8   m=256   fp32  s_i * N(0,1), s_i ~ U[0.5, 2]
  gpt2small   d=124,439,808 n=16 m=1024  bf16  Student-t(nu=3)
  sweep       d=1e9        n=2   m in {8,64,512,4096}  fp32  N(0,1)
  leastsq     n=8 machines, A_i 2048 x 8192, rows ~ N(0, diag(lambda)/d),
              lambda_k = k^-1.5, b_i = A_i x* + 0.01 N(0,1), x* ~ N(0, I)
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    d: int
    n: int
    m: tuple
    dtype: str          # "f32" | "bf16"
    dist: str           # "normal" | "scaled_normal" | "student_t3"


WORKLOADS = {
    "tiny": Workload("tiny", 4096, 4, (16,), "f32", "normal"),
    "resnet50": Workload("resnet50", 25_557_032, 8, (256,), "f32", "scaled_normal"),
    "gpt2small": Workload("gpt2small", 124_439_808, 16, (1024,), "bf16", "student_t3"),
    "sweep": Workload("sweep", 1_000_000_000, 2, (8, 64, 512, 4096), "f32", "normal"),
}


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def gradients(n: int, d: int, seed: int = 0, dist: str = "normal", dtype: str = "f32",
              device="cpu", ld: int | None = None) -> torch.Tensor:
    """G[n, d] (a view into an [n, ld] allocation when ld > d), one row per simulated machine.

    dist = "normal":        g ~ N(0,1)
    dist = "scaled_normal": g_i = s_i N(0,1), s_i ~ U[0.5, 2] per machine
    dist = "student_t3":    g = z0 / sqrt((z1^2 + z2^2 + z3^2) / 3), heavy-tailed
    dtype = "bf16" rounds (to nearest even) once, at the end.
    """
    ld = d if ld is None else ld
    assert ld >= d
    gen = _gen(seed, device)
    store = torch.zeros((n, ld), dtype=torch.float32, device=device)
    G = store[:, :d]
    scales = None
    if dist == "scaled_normal":
        scales = 0.5 + 1.5 * torch.rand(n, generator=gen, device=device)
    piece = 1 << 24
    for i in range(n):
        row = G[i]
        if dist in ("normal", "scaled_normal"):
            for s in range(0, d, 1 << 26):
                row[s:min(s + (1 << 26), d)].normal_(generator=gen)
            if scales is not None:
                row.mul_(scales[i])
        elif dist == "student_t3":
            for s in range(0, d, piece):
                e = min(s + piece, d)
                z = torch.randn((4, e - s), generator=gen, device=device)
                chi = (z[1] * z[1] + z[2] * z[2] + z[3] * z[3]) / 3.0
                row[s:e] = z[0] / torch.sqrt(chi)
        else:
            raise ValueError(dist)
    if dtype == "bf16":
        store16 = store.to(torch.bfloat16)
        return store16[:, :d]
    if dtype != "f32":
        raise ValueError(dtype)
    return G


def workload_gradients(name: str, seed: int = 0, device="cpu") -> torch.Tensor:
    w = WORKLOADS[name]
    return gradients(w.n, w.d, seed=seed, dist=w.dist, dtype=w.dtype, device=device)


def to_oracle_array(G: torch.Tensor) -> np.ndarray:
    """Host copy of G for the oracle: float32 stays float32; bf16 becomes its uint16 bit patterns."""
    G = G.detach()
    if G.dtype == torch.bfloat16:
        return G.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    return G.contiguous().cpu().numpy()


@dataclass
class LeastSquares:
    A: torch.Tensor      # [n, rows, d] fp32
    b: torch.Tensor      # [n, rows]    fp32
    x_star: torch.Tensor  # [d]          fp32
    lam: torch.Tensor    # [d] spectrum


def least_squares(n: int = 8, rows: int = 2048, d: int = 8192, seed: int = 0, decay: float = 1.5,
                  noise: float = 0.01, device="cpu") -> LeastSquares:
    """Distributed least squares with a power-law spectrum lambda_k = k^-decay (k = 1..d)."""
    gen = _gen(seed, device)
    k = torch.arange(1, d + 1, dtype=torch.float64, device=device)
    lam = k.pow(-decay)
    col_scale = torch.sqrt(lam / d).to(torch.float32)
    x_star = torch.randn(d, generator=gen, device=device)
    A = torch.empty((n, rows, d), dtype=torch.float32, device=device)
    b = torch.empty((n, rows), dtype=torch.float32, device=device)
    for i in range(n):
        A[i].normal_(generator=gen)
        A[i].mul_(col_scale)
        eps = torch.randn(rows, generator=gen, device=device)
        b[i] = (A[i].double() @ x_star.double()).float() + noise * eps
    return LeastSquares(A, b, x_star, lam)


def lipschitz_constant(A: torch.Tensor, iters: int = 100) -> float:
    """Largest eigenvalue of (1/n) sum_i A_i^T A_i / rows by a fixed fp64 power iteration."""
    n, rows, d = A.shape
    v = torch.ones(d, dtype=torch.float64, device=A.device) / np.sqrt(d)
    lam = 0.0
    for _ in range(iters):
        w = torch.zeros_like(v)
        for i in range(n):
            Ai = A[i].double()
            w += Ai.T @ (Ai @ v)
        w /= (n * rows)
        lam = float(torch.linalg.norm(w))
        v = w / lam
    return lam


def gossip_matrix(topology: str, n: int) -> np.ndarray:
    """A network for the decentralised variant, given as its gossip matrix W (n x n float64, symmetric,
    doubly stochastic, W[i][l] = 0 unless machines i and l are neighbours or i = l).

    "ring":     machine i talks to i-1 and i+1 (mod n); weights 1/3 on each neighbour and on itself
                (for n = 2 the two neighbours coincide: 1/2 and 1/2; n = 1: the 1 x 1 identity).
    "torus":    machines on an a x b grid with wrap-around, a the largest divisor of n not above
                sqrt(n); weight 1/5 on each of the four grid neighbours, the rest on itself
                (coinciding neighbours add up).
    "complete": every machine talks to every other: all weights 1/n (one round reaches the mean).
    """
    W = np.zeros((n, n), dtype=np.float64)
    if topology == "complete":
        W[:] = 1.0 / n
        return W
    if topology == "ring":
        for i in range(n):
            for l in ((i - 1) % n, (i + 1) % n):
                W[i, l] += 1.0 / 3.0
    elif topology == "torus":
        a = max(k for k in range(1, int(np.sqrt(n)) + 1) if n % k == 0)
        b = n // a
        for i in range(n):
            r, c = divmod(i, b)
            for l in (((r - 1) % a) * b + c, ((r + 1) % a) * b + c, r * b + (c - 1) % b, r * b + (c + 1) % b):
                W[i, l] += 1.0 / 5.0
    else:
        raise ValueError(topology)
    for i in range(n):
        W[i, i] = 0.0
        W[i, i] = 1.0 - W[i].sum()
    return W
