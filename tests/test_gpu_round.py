"""GPU parity of project / aggregate / reconstruct against the oracle, through the C ABI.

Bars: |p_gpu - p_oracle| <= 1e-4 ||g_i||_2 for every message entry; reconstruction relative
L2 error <= 1e-4.  Small and medium cases are compared element by element; at the full
sizes of the evaluation workloads the oracle computes sampled outputs (all of d for a few
(i, j); all of m for sampled coordinate blocks).
"""
import numpy as np
import pytest
import torch

import core_inputs
import oracle
from helpers import P_TOL, REC_TOL, oracle_project_entry, rel_l2, row_norms

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def core_mod():
    import paper_2309_13307_b200 as core_mod
    core_mod.lib()
    return core_mod


def check_round(core_mod, G: torch.Tensor, m: int, seed: int = 1, t: int = 0):
    """Full element-wise comparison of every stage of one round."""
    Gh = core_inputs.to_oracle_array(G)
    n, d = G.shape
    ctx = core_mod.Core(seed, d, m)
    ctx.core_set_round(t)
    P = ctx.core_project(G)
    pbar = ctx.core_aggregate(P)
    gt = ctx.core_reconstruct(pbar)
    Po, pbaro, gto = oracle.core_round(seed, t, m, Gh)
    norms = row_norms(Gh)
    dP = np.abs(P.cpu().numpy().astype(np.float64) - Po)
    assert (dP <= P_TOL * norms[:, None] + 1e-30).all(), float((dP / norms[:, None]).max())
    assert np.abs(pbar.cpu().numpy() - pbaro).max() <= P_TOL * norms.mean() + 1e-30
    assert rel_l2(gt.cpu().numpy(), gto) <= REC_TOL
    # the fused entry point gives the same answer and advances the round
    pbar2, gt2 = ctx.core_round(G)
    assert ctx.core_get_round() == t + 1
    assert torch.equal(pbar2, pbar) and torch.equal(gt2, gt)
    assert core_mod.core_device_status() == 0        # no bounded wait of the tensor-memory kernel ran out
    # reconstruction alone, from the oracle's message (isolates the second kernel)
    ctx.core_set_round(t)
    gt3 = ctx.core_reconstruct(torch.from_numpy(pbaro.astype(np.float32)).cuda())
    assert rel_l2(gt3.cpu().numpy(), gto) <= REC_TOL
    return ctx


def test_tiny_workload(core_mod):
    w = core_inputs.WORKLOADS["tiny"]
    G = core_inputs.workload_gradients("tiny", seed=0, device="cuda")
    check_round(core_mod, G, w.m[0], seed=1, t=0)


@pytest.mark.parametrize("d", [1, 3, 4, 5, 8, 4095, 4096, 4097, 10007])
@pytest.mark.parametrize("m,n", [(1, 1), (3, 4), (16, 4)])
def test_ragged_sizes(core_mod, d, m, n):
    G = core_inputs.gradients(n, d, seed=d + m, device="cuda")
    check_round(core_mod, G, m, seed=3, t=2)


@pytest.mark.parametrize("n,m,d,dtype,dist", [
    (2, 8, 200_003, "f32", "normal"),            # short-vector plans: 32-block tiles, vectors shared among warps
    (2, 8, 1_300_003, "f32", "normal"),          # long-vector plans: several large tiles per CTA column, ragged tail
    (8, 64, 400_003, "bf16", "scaled_normal"),
    (8, 64, 65_537, "f32", "scaled_normal"),
    (16, 40, 33_000, "bf16", "student_t3"),
    (17, 5, 20_001, "f32", "normal"),            # more than one machine group
    (3, 600, 9_001, "bf16", "normal"),           # more vectors than one CTA row holds
    (5, 1030, 8_200, "f32", "normal"),
    (2, 5000, 4_100, "f32", "normal"),           # more vectors than one reconstruction table chunk (2048)
    (1, 2049, 1_000, "bf16", "normal"),
    (40, 3, 4_097, "bf16", "student_t3"),        # three machine groups
    (16, 130, 20_003, "bf16", "student_t3"),     # 9..16 machines and m >= 64: the tensor-core projection
    (11, 64, 9_001, "f32", "scaled_normal"),
    (9, 200, 70_000, "f32", "normal"),
    (25, 72, 3_000, "f32", "normal"),            # two tensor-core passes: 16 machines, then 9
    (16, 256, 20_003, "bf16", "student_t3"),     # 9..16 machines and m >= 96: the tensor-memory (tcgen05) projection
    (12, 1024, 5_003, "f32", "normal"),          # more CTA rows than coordinate tiles per column
    (16, 384, 40_001, "f32", "scaled_normal"),
    (10, 200, 300, "bf16", "normal"),            # a single ragged tile; last CTA row 72 of 128 vectors
    (41, 128, 2_049, "f32", "normal"),           # a tensor-memory pass of 32 machines, then one of 9
    (32, 256, 30_011, "f32", "scaled_normal"),   # 32 machines in one pass (N = 32 of the instruction), fp32: two-stage ring
    (32, 256, 30_011, "bf16", "student_t3"),     # the same with one gradient plane and a three-stage ring
    (50, 130, 9_001, "f32", "normal"),           # 32 + 18 machines
    (64, 1024, 5_003, "bf16", "normal"),         # 64 machines in one pass (N = 64, 256 vectors per CTA)
    (50, 256, 30_011, "f32", "normal"),          # 50 machines, fp32: N = 64 with a two-stage ring
    (33, 512, 9_001, "f32", "scaled_normal"),    # 33 machines: N = 64 with 31 empty columns
    (64, 128, 9_001, "bf16", "normal"),          # 64 machines, 128 vectors: two passes of 32
    (70, 256, 9_001, "bf16", "student_t3"),      # 64 + 6
    (17, 96, 70_001, "bf16", "scaled_normal"),   # 17 machines: N = 32 with 15 empty columns
    (16, 456, 30_001, "f32", "normal"),          # two groups of 128 vectors per CTA, second CTA row 200 of 256 full
    (20, 456, 30_001, "bf16", "student_t3"),     # the same with N = 32
])
def test_medium_sizes(core_mod, n, m, d, dtype, dist):
    G = core_inputs.gradients(n, d, seed=11, dist=dist, dtype=dtype, device="cuda")
    check_round(core_mod, G, m, seed=5, t=1)


@pytest.mark.parametrize("n,d,m", [(3, 5003, 7), (10, 3001, 70), (13, 3001, 256)])   # scalar, warp-level and tcgen05 projection
def test_unaligned_rows_and_leading_dimension(core_mod, n, d, m):
    for dtype in ("f32", "bf16"):
        # ld > d with an odd stride, and a base pointer that is not 16-byte aligned
        store = core_inputs.gradients(n, d + 1, seed=2, dtype=dtype, device="cuda", ld=d + 9)
        G = store[:, 1:]
        assert G.shape == (n, d) and G.stride(0) == d + 9
        check_round(core_mod, G, m, seed=8, t=0)


@pytest.mark.parametrize("n,m", [(8, 64), (16, 256)])                 # scalar and tcgen05 projection
def test_bitwise_reproducible(core_mod, n, m):
    G = core_inputs.gradients(n, 300_000, seed=4, device="cuda")
    ctx = core_mod.Core(1, G.shape[1], m)
    a = ctx.core_round(G)
    ctx.core_set_round(0)
    b = ctx.core_round(G)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


def test_device_status_word(core_mod):
    import ctypes
    assert core_mod.core_device_status() == 0
    assert core_mod.lib().core_device_status(None) == -1        # CORE_EINVAL


@pytest.mark.parametrize("n,m,dtype", [
    (2, 8, "f32"), (4, 40, "bf16"), (8, 64, "f32"),       # scalar projection
    (10, 70, "f32"), (12, 72, "bf16"),                    # warp-level tensor-core projection
    (16, 256, "bf16"), (9, 128, "f32"),                   # tcgen05 projection
    (32, 128, "f32"), (27, 256, "bf16"),                  # tcgen05 projection, 32 machines per pass
    (64, 256, "bf16"), (40, 512, "f32"),                  # tcgen05 projection, 64 machines per pass
])
def test_unit_vectors_read_the_generator_back(core_mod, n, m, dtype):
    """Machine i holds the unit vector e_k(i): its message is p_ij = xi_j[k(i)], and every other term of
    the sum is an exact zero, so the scalar projection must return the generator's own fp32 values bit for
    bit.  On the tensor-core paths the tail of a split value is itself cut to tf32, which leaves 2^-21 of
    the value.  Likewise pbar = e_j reconstructs xi_j / m, bit for bit."""
    d, seed, t = 70_001, 6, 3
    ks = [(i * 7919 + 5) % d for i in range(n)]
    ks[0], ks[-1] = 0, d - 1                               # first block, ragged last block
    G = torch.zeros((n, d), dtype=torch.float32, device="cuda")
    for i, k in enumerate(ks):
        G[i, k] = 1.0
    if dtype == "bf16":
        G = G.to(torch.bfloat16)
    ctx = core_mod.Core(seed, d, m)
    ctx.core_set_round(t)
    P = ctx.core_project(G)
    assert core_mod.core_device_status() == 0
    scalar = n <= 8
    for j in sorted({0, 1, m // 2, m - 1}):
        z = ctx.core_debug_gaussians(j, 0, (d + 3) // 4).reshape(-1)      # xi_j[0 .. 4 ceil(d/4))
        for i, k in enumerate(ks):
            got, want = P[i, j].item(), z[k].item()
            assert got == want if scalar else abs(got - want) <= 2.0 ** -20 * abs(want), (i, j, k, got, want)
    for j in sorted({0, m - 1}):
        pbar = torch.zeros(m, dtype=torch.float32, device="cuda")
        pbar[j] = 1.0
        gt = ctx.core_reconstruct(pbar)
        z = ctx.core_debug_gaussians(j, 0, (d + 3) // 4).reshape(-1)[:d]
        assert torch.equal(gt, z * torch.tensor(1.0 / m, dtype=torch.float32, device="cuda")), j


def test_round_index_and_seed_change_the_vectors(core_mod):
    G = core_inputs.gradients(2, 4096, seed=4, device="cuda")
    base = core_mod.Core(1, 4096, 8).core_project(G)
    other = core_mod.Core(1, 4096, 8)
    other.core_set_round(1)
    assert not torch.equal(base, other.core_project(G))
    assert not torch.equal(base, core_mod.Core(2, 4096, 8).core_project(G))


def test_host_round_matches_oracle_and_device_round(core_mod):
    n, d, m = 4, 3_000_017, 16       # several slabs would need more; here one ragged slab ...
    G = core_inputs.gradients(n, d, seed=6, device="cuda")
    Gh = G.cpu().pin_memory()
    ctx = core_mod.Core(2, d, m)
    pbar_h = torch.empty(m, dtype=torch.float32).pin_memory()
    gt_h = torch.empty(d, dtype=torch.float32).pin_memory()
    ctx.core_round_host(Gh, pbar_h, gt_h)
    assert ctx.core_get_round() == 1
    ctx.core_set_round(0)
    pbar_d, gt_d = ctx.core_round(G)
    norm = float(row_norms(Gh.numpy()).mean())
    assert np.abs(pbar_h.numpy() - pbar_d.cpu().numpy()).max() <= P_TOL * norm
    # sampled oracle values of the message, then the reconstruction from the oracle's message
    for j in (0, m - 1):
        want = np.mean([oracle_project_entry(2, 0, j, Gh.numpy()[i]) for i in range(n)])
        assert abs(float(pbar_h[j]) - want) <= P_TOL * norm
    k0 = 2_999_900
    want = oracle.reconstruct_slice(2, 0, pbar_h.numpy().astype(np.float64), k0, d)
    assert rel_l2(gt_h.numpy()[k0:], want) <= REC_TOL
    assert rel_l2(gt_h.numpy(), gt_d.cpu().numpy()) <= REC_TOL


@pytest.mark.parametrize("m", [8, 128])      # scalar and tcgen05 projection (slabs start at non-zero blocks)
def test_host_round_many_slabs(core_mod, m):
    # bf16, 16 machines: slabs of 2^21 coordinates, so d = 5e6 + 3 takes three slabs
    n, d = 16, 5_000_003
    G = core_inputs.gradients(n, d, seed=3, dtype="bf16", dist="student_t3", device="cuda")
    Gh = G.cpu()
    ctx = core_mod.Core(4, d, m)
    pbar_h = torch.empty(m, dtype=torch.float32)
    gt_h = torch.empty(d, dtype=torch.float32)
    ctx.core_round_host(Gh, pbar_h, gt_h)
    ctx.core_set_round(0)
    pbar_d, gt_d = ctx.core_round(G)
    bits = core_inputs.to_oracle_array(Gh)
    norm = float(row_norms(bits).mean())
    assert np.abs(pbar_h.numpy() - pbar_d.cpu().numpy()).max() <= P_TOL * norm
    want = np.mean([oracle_project_entry(4, 0, 3, bits[i]) for i in range(n)])
    assert abs(float(pbar_h[3]) - want) <= P_TOL * norm
    for k0, k1 in [(0, 64), (2_097_100, 2_097_200), (d - 50, d)]:
        want = oracle.reconstruct_slice(4, 0, pbar_h.numpy().astype(np.float64), k0, k1)
        assert rel_l2(gt_h.numpy()[k0:k1], want) <= REC_TOL


@pytest.mark.parametrize("kind,n,m,dtype", [(2, 5, 128, "f32"), (2, 8, 256, "bf16"), (2, 3, 40, "f32"), (2, 20, 33, "bf16"),
                                          (0, 16, 256, "bf16"), (0, 12, 128, "f32"), (1, 16, 256, "f32")])
def test_each_projection_kernel_on_shapes_the_default_would_not_give_it(core_mod, kind, n, m, dtype):
    """The tensor-memory kernel with few machines and few vectors, the scalar and the warp-level kernels on
    shapes that normally go to the tensor-memory kernel: all must meet the same bars."""
    from paper_2309_13307_b200 import binding
    G = core_inputs.gradients(n, 50_021, seed=21, dtype=dtype, device="cuda")
    binding.core_debug_force_project_kernel(kind)
    try:
        plan = binding.core_debug_project_plan(n, m, 50_021, binding.CORE_BF16 if dtype == "bf16" else binding.CORE_F32,
                                               torch.cuda.get_device_properties(0).multi_processor_count)
        assert (plan["tj"] == 32 and plan["tq"] == 8 and plan["tile_q"] == 64) == (kind == 2)   # the tcgen05 geometry
        check_round(core_mod, G, m, seed=9, t=4)
    finally:
        binding.core_debug_force_project_kernel(-1)
    assert core_mod.lib().core_debug_force_project_kernel(3) == -1


# ---- full-size workloads, sampled ---------------------------------------------------

def sampled_full_size(core_mod, name: str, m: int, js, machines, seed=1, t=0):
    w = core_inputs.WORKLOADS[name]
    G = core_inputs.workload_gradients(name, seed=0, device="cuda")
    ctx = core_mod.Core(seed, w.d, m)
    ctx.core_set_round(t)
    P = ctx.core_project(G).cpu().numpy()
    for i in machines:
        row = core_inputs.to_oracle_array(G[i:i + 1])[0]
        norm = float(row_norms(row[None, :])[0])
        for j in js:
            want = oracle_project_entry(seed, t, j, row)
            assert abs(float(P[i, j]) - want) <= P_TOL * norm, (i, j, float(P[i, j]), want, norm)
    del G
    # reconstruction from a seeded synthetic message, on sampled coordinate ranges
    pbar = core_inputs.gradients(1, m, seed=99).numpy()[0]
    gt = ctx.core_reconstruct(torch.from_numpy(pbar).cuda())
    rng = np.random.default_rng(5)
    starts = [0, w.d - 37] + [int(s) for s in rng.integers(0, w.d - 64, size=6)]
    for k0 in starts:
        k1 = min(k0 + 37, w.d)
        want = oracle.reconstruct_slice(seed, t, pbar.astype(np.float64), k0, k1)
        assert rel_l2(gt[k0:k1].cpu().numpy(), want) <= REC_TOL
    # a property that holds at any size: <gbar, gtilde> = (1/m) sum_j pbar_j^2 needs the true
    # message, so check the cheaper one: every coordinate was written (no NaN canary left)
    assert bool(torch.isfinite(gt).all())


def test_resnet50_sized(core_mod):
    sampled_full_size(core_mod, "resnet50", 256, js=(0, 255), machines=(0, 7))


def test_gpt2small_sized_bf16(core_mod):
    sampled_full_size(core_mod, "gpt2small", 1024, js=(511,), machines=(0, 15))


@pytest.mark.parametrize("name,m", [("resnet50", 256), ("gpt2small", 1024)])
def test_full_size_round_keeps_the_inner_product(core_mod, name, m):
    """A property that holds at any size and involves every coordinate and every vector:
    <gbar, gtilde> = (1/m) sum_j pbar_j <gbar, xi_j> = (1/m) sum_j pbar_j^2, with gbar the mean
    gradient.  Projection and reconstruction must have regenerated the same vectors for it to hold."""
    w = core_inputs.WORKLOADS[name]
    G = core_inputs.workload_gradients(name, seed=0, device="cuda")
    ctx = core_mod.Core(1, w.d, m)
    pbar, gt = ctx.core_round(G)
    assert core_mod.core_device_status() == 0
    lhs = 0.0
    step = 1 << 22
    for k0 in range(0, w.d, step):                      # fp64 in chunks: the operands are large
        gbar = G[:, k0:k0 + step].to(torch.float64).mean(dim=0)
        lhs += float((gbar * gt[k0:k0 + step].to(torch.float64)).sum())
    rhs = float((pbar.to(torch.float64) ** 2).sum()) / m
    # fp32 accumulation leaves about 1e-7 of ||gtilde|| ~ ||gbar|| sqrt(d / m) in gtilde
    assert abs(lhs - rhs) <= 5e-3 * rhs, (lhs, rhs)


@pytest.mark.parametrize("m", [8, 64, 512, 4096])      # every launch plan of the sweep (tj = 2, 16, 128, 256)
def test_sweep_sized(core_mod, m):
    sampled_full_size(core_mod, "sweep", m, js=(m - 1,), machines=(1,))
