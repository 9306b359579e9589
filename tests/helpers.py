"""Shared helpers of the GPU parity tests (no arithmetic of the method lives here)."""
import math
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

import oracle

P_TOL = 1e-4        # |p_gpu - p_oracle| <= P_TOL * ||g_i||_2
REC_TOL = 1e-4      # ||gt_gpu - gt_oracle||_2 <= REC_TOL * ||gt_oracle||_2


def host_threads() -> int:
    return max(1, min(32, os.cpu_count() or 1))


def oracle_project_entry(seed, t, j, g_row: np.ndarray, threads: int | None = None) -> float:
    """<g, xi_j> by the oracle, the coordinate range cut into pieces that run on several host
    threads (the oracle call releases the GIL); the pieces are added in fp64."""
    d = g_row.shape[0]
    threads = threads or host_threads()
    piece = max(4096, (d // threads + 3) // 4 * 4)
    cuts = list(range(0, d, piece)) + [d]
    oracle.lib()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        parts = list(ex.map(lambda ab: oracle.project_slice(seed, t, j, g_row, ab[0], ab[1]),
                            zip(cuts[:-1], cuts[1:])))
    return math.fsum(parts)


def row_norms(G: np.ndarray) -> np.ndarray:
    if G.dtype == np.uint16:
        G = (G.astype(np.uint32) << 16).view(np.float32)
    return np.sqrt((G.astype(np.float64) ** 2).sum(axis=1))


def rel_l2(a: np.ndarray, b: np.ndarray) -> float:
    a = a.astype(np.float64)
    b = b.astype(np.float64)
    den = math.sqrt(float((b * b).sum()))
    return math.sqrt(float(((a - b) ** 2).sum())) / (den if den > 0 else 1.0)
