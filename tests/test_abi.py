"""The C-ABI library builds, loads, and exports every symbol include/core.h declares (CPU only:
nothing here launches a kernel)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "core.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(core_[a-z0-9_]+)\s*\(", text)))


@pytest.fixture(scope="module")
def library():
    from paper_2309_13307_b200 import build
    return ctypes.CDLL(build.build())


def test_header_declares_the_round_entry_points():
    names = declared_symbols()
    for required in ("core_init", "core_project", "core_aggregate", "core_reconstruct", "core_gd_step",
                     "core_round", "core_round_host", "core_destroy"):
        assert required in names


def test_library_exports_every_declared_symbol(library):
    for name in declared_symbols():
        assert hasattr(library, name), name


def test_binding_covers_every_declared_symbol():
    from paper_2309_13307_b200 import binding
    assert sorted(binding.exported_symbols()) == declared_symbols()


def test_host_side_argument_checks(library):
    # these return before touching the device
    assert library.core_init(None, ctypes.c_uint64(1), ctypes.c_int64(8), ctypes.c_int32(2)) == -1
    h = ctypes.c_void_p()
    assert library.core_init(ctypes.byref(h), ctypes.c_uint64(1), ctypes.c_int64(0), ctypes.c_int32(2)) == -1
    assert library.core_init(ctypes.byref(h), ctypes.c_uint64(1), ctypes.c_int64(8), ctypes.c_int32(0)) == -1
    assert h.value is None
    library.core_strerror.restype = ctypes.c_char_p
    assert library.core_strerror(-1) == b"invalid argument"
    assert library.core_destroy(None) == -1
    assert library.core_set_round(None, 3) == -1


def test_project_plans_are_consistent():
    """Launch geometry (host logic): the thread grid covers all m vectors and all tiles of d,
    the per-thread stepping divides a tile, and the shared memory fits an SM."""
    from paper_2309_13307_b200 import binding
    for n in (1, 2, 3, 4, 8, 16, 40, 70):
        for m in (1, 2, 8, 64, 511, 512, 1030, 4096, 100_000):
            for d in (1, 4097, 25_557_032, 1_000_000_000):
                for dtype in (binding.CORE_F32, binding.CORE_BF16):
                    p = binding.core_debug_project_plan(n, m, d, dtype, 148)
                    tensor_memory = (p["tj"], p["tq"], p["tile_q"]) == (32, 8, 64)
                    assert p["nb"] >= min(n, 16) and p["nb"] in (1, 2, 4, 8, 16, 32, 64)
                    assert p["nb"] <= 16 or (tensor_memory and n > 16 and m >= 96)
                    assert p["nb"] <= 32 or (n > 32 and p["jt"] == 8)        # 64 machines need 256 vectors per CTA
                    assert p["tj"] * p["tq"] == 256
                    assert p["tile_q"] % (p["tq"] * p["uq"]) == 0
                    assert p["grid_y"] * p["tj"] * p["jt"] >= m
                    assert p["tiles"] * 4 * p["tile_q"] >= d > (p["tiles"] - 1) * 4 * p["tile_q"]
                    assert 1 <= p["grid_x"] <= p["tiles"]
                    assert p["smem"] <= 227 * 1024
                    if not tensor_memory:
                        assert p["smem"] >= 256 * p["nb"] * p["jt"] * 4      # room for the final reduction
