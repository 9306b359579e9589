"""GPU parity of the common random generator against the oracle (through the C ABI).

Bars: Philox words bit-exact; Gaussians within 4e-6 absolute, extremes included.
"""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu

GAUSS_TOL = 4e-6


@pytest.fixture(scope="module")
def core_mod():
    import paper_2309_13307_b200 as core_mod
    core_mod.lib()
    return core_mod


def as_u32(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32)


@pytest.mark.parametrize("seed,t,j,q0,nq", [
    (1, 0, 0, 0, 1 << 20),
    (1, 0, 15, 0, 4099),
    (0xDEADBEEFCAFEF00D, 7, 4095, (1 << 32) - 1000, 2000),      # crosses the high counter word
    (5, 2**32 - 1, 2**32 - 1, (1 << 40) + 3, 1 << 18),
    (2**64 - 1, 3, 1023, 249_999_000, 1 << 20),
])
def test_philox_words_bit_exact(core_mod, seed, t, j, q0, nq):
    ctx = core_mod.Core(seed, 16, 1)
    ctx.core_set_round(t)
    got = as_u32(ctx.core_debug_philox(j, q0, nq))
    want = oracle.xi_words_range(seed, t, j, q0, q0 + nq)
    assert np.array_equal(got, want)


def test_gaussians_window_within_tolerance(core_mod):
    total = 0
    for seed, t, j, q0, nq in [(1, 0, 0, 0, 1 << 20), (9, 4, 255, (1 << 32) - 4096, 1 << 19),
                               (77, 1, 1023, 31_000_000, 1 << 20)]:
        ctx = core_mod.Core(seed, 16, 1)
        ctx.core_set_round(t)
        got = ctx.core_debug_gaussians(j, q0, nq).cpu().numpy().astype(np.float64)
        want = oracle.box_muller_many(oracle.xi_words_range(seed, t, j, q0, q0 + nq))
        assert np.abs(got - want).max() <= GAUSS_TOL
        total += got.size
    assert total >= 10_000_000


def test_box_muller_every_radius_and_every_angle(core_mod):
    """All 2^23 radius inputs (at the angles where |cos| and |sin| peak) and all 2^23 angle
    inputs (at the largest radius), so the extremes of both are covered."""
    ctx = core_mod.Core(1, 16, 1)
    k = np.arange(1 << 23, dtype=np.uint32) << np.uint32(9)
    worst = 0.0
    # lanes: (radius word, angle word, radius word, angle word)
    cases = [
        (k, np.zeros_like(k), k, np.full_like(k, 0x40000000)),              # every radius; angle ~0 and ~pi/2
        (np.zeros_like(k), k, np.full_like(k, 0xFFFFFFFF), k),              # every angle; largest / smallest radius
        (np.full_like(k, 0x00000200), k, np.full_like(k, 0x80000000), k),   # every angle; r ~ 5.58 and r ~ 1.18
    ]
    for lanes in cases:
        words = np.stack(lanes, axis=1)
        got = ctx.core_debug_box_muller(torch.from_numpy(words.view(np.int32)).cuda()).cpu().numpy()
        want = oracle.box_muller_many(words)
        worst = max(worst, float(np.abs(got.astype(np.float64) - want).max()))
    assert worst <= GAUSS_TOL, worst
