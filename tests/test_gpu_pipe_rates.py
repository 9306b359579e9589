"""Instruction-rate probes behind the round kernels' roofline (through the C ABI).

The round kernels are bound by instruction issue.  Their "alu" peak rests on three measured facts
about this GPU, asserted here on the device the tests run on (cycle counts: independent of the clock):
  * a 32x32->64-bit integer multiply occupies a scheduler for 4 cycles per warp instruction
    (32 lanes per clock per SM), against 1 for an fp32 multiply-add and 2 for a logic or a packed op;
  * other instructions do not hide behind it: a mixed stream costs about the sum of its parts;
  * the fp64 unit can produce the high word of the product exactly (checksums agree).
Run with ``-s`` to print the whole table (the source of profiles/pipe_rates.md).
"""
import pytest

pytestmark = pytest.mark.gpu

NAMES = ("wide", "ffma", "ffma2", "lop3", "mufu", "dfma", "imad")


@pytest.fixture(scope="module")
def core_mod():
    import paper_2309_13307_b200 as core_mod
    core_mod.lib()
    return core_mod


@pytest.fixture(scope="module")
def table(core_mod):
    from paper_2309_13307_b200 import binding
    kinds = binding.core_debug_pipe_kinds()
    rows = {}
    for kind in range(kinds):
        mix = binding.core_debug_pipe_mix(kind)
        for wps in (4, 8):
            cyc, chk = binding.core_debug_pipe_cycles(kind, wps, 2048, seed=3)
            rows[(kind, wps)] = (mix, cyc, chk)
    print()
    print("kind  warps/sched  body                                     cycles/body/warp")
    for (kind, wps), (mix, cyc, chk) in rows.items():
        body = " + ".join(f"{c} {n}" for c, n in zip(mix, NAMES) if c) or f"Philox rounds 2..9 x 4 counters, multiply mode {kind - (kinds - 3)}"
        print(f"{kind:4d}  {wps:11d}  {body:40s} {cyc:8.2f}   checksum {chk:08x}")
    return rows, kinds


def test_per_instruction_costs(table):
    """Cycles a scheduler spends per warp instruction when a loop holds only that class."""
    rows, _ = table
    for wps in (4, 8):
        per = {name: rows[(kind, wps)][1] / count for kind, name, count in
               [(0, "wide", 16), (1, "ffma", 64), (2, "ffma2", 32), (3, "lop3", 64), (4, "mufu", 16), (5, "dfma", 32),
                (6, "imad", 32)]}
        assert 3.6 <= per["wide"] <= 4.6, per          # the multiplier behind mul.wide.u32: 32 lanes / clock / SM
        assert 0.95 <= per["ffma"] <= 1.2, per         # 128 lanes / clock / SM
        for name in ("ffma2", "lop3", "dfma", "imad"):
            assert 1.8 <= per[name] <= 2.4, (name, per)
        assert 7.0 <= per["mufu"] <= 9.0, per


def test_philox_rounds_alone(table):
    """Rounds 2..9 of one counter (16 wide multiplies, 18 logic ops after hoisting): what the generator's
    integer half costs a scheduler per warp and counter when nothing else runs."""
    rows, kinds = table
    for wps in (4, 8):
        per_counter = rows[(kinds - 3, wps)][1] / 4
        assert 64.0 <= per_counter <= 84.0, per_counter


def test_other_work_does_not_hide_behind_the_wide_multiply(table):
    rows, _ = table
    alone = rows[(0, 8)][1]
    assert rows[(7, 8)][1] >= alone + 0.5 * 16          # + 16 fp32 multiply-adds
    assert rows[(8, 8)][1] >= alone + 0.5 * 32          # + 32
    assert rows[(11, 8)][1] >= alone + 0.5 * 32         # + 32 logic ops


def test_fp64_route_gives_the_same_words(table):
    rows, kinds = table
    sums = {rows[(k, 4)][2] for k in range(kinds - 3, kinds)}
    assert len(sums) == 1, sums
