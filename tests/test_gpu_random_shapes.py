"""Seeded random shapes against the oracle (through the C ABI): machine counts on both sides of every
kernel choice (scalar, warp-level, tensor-memory with 128 or 256 vectors per CTA and 16, 32 or 64 machines
per pass), vector counts around the CTA-row sizes, ragged lengths, unaligned rows and padded leading
dimensions, both gradient types.  Same bars as the other round tests."""
import random

import pytest
import torch

import core_inputs
from test_gpu_round import check_round, core_mod  # noqa: F401  (fixture)

pytestmark = pytest.mark.gpu

NS = [1, 2, 3, 5, 8, 9, 16, 17, 31, 32, 33, 48, 50, 64, 65, 70]
MS = [1, 5, 16, 63, 64, 95, 96, 127, 128, 129, 192, 255, 256, 257, 384, 449, 512, 1000, 1024]
DS = [1, 3, 33, 256, 257, 1000, 4097, 9001, 20003]


def cases(count=36, seed=7):
    rng = random.Random(seed)
    out = []
    while len(out) < count:
        n, m, d = rng.choice(NS), rng.choice(MS), rng.choice(DS)
        if n * m * d > 3e8:                      # keeps the oracle's share to about a second per case
            continue
        out.append((n, m, d, rng.choice(["f32", "bf16"]), rng.choice([0, 0, 1, 4]), rng.choice([0, 0, 3, 8]),
                    rng.choice(["normal", "scaled_normal", "student_t3"]), rng.randrange(1 << 40), rng.randrange(5)))
    return out


@pytest.mark.parametrize("n,m,d,dtype,offset,pad,dist,seed,t", cases())
def test_random_shape(core_mod, n, m, d, dtype, offset, pad, dist, seed, t):  # noqa: F811
    store = core_inputs.gradients(n, d + offset, seed=n + m + d, dist=dist, dtype=dtype, device="cuda",
                                  ld=d + offset + pad)
    check_round(core_mod, store[:, offset:], m, seed=seed, t=t)
