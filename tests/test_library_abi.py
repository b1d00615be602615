"""The C-ABI library builds, loads, and exports every symbol that include/fbsr.h declares
(no compute calls: this runs without a GPU), and host-side logic behaves."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2504_20634_b200 import build
    return ctypes.CDLL(build.build())


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "fbsr.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fbsr_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_expected_entry_points():
    names = declared_symbols()
    for must in ("fbsr_round", "fbsr_round_bits", "fbsr_round_stats", "fbsr_sgd_update", "fbsr_adam_update",
                 "fbsr_accumulate", "fbsr_round_host", "fbsr_status_string", "fbsr_version"):
        assert must in names


def test_every_declared_symbol_is_exported(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_host_side_queries(lib):
    lib.fbsr_tile_elements.restype = ctypes.c_size_t
    lib.fbsr_status_string.restype = ctypes.c_char_p
    lib.fbsr_stats_workspace_bytes.restype = ctypes.c_size_t
    for k in range(1, 17):
        tile = lib.fbsr_tile_elements(k)
        E = 4 * (32 // k)
        assert tile % 256 == 0 and tile % E == 0 and tile >= 1024
    assert lib.fbsr_tile_elements(0) == 0 and lib.fbsr_tile_elements(17) == 0
    assert lib.fbsr_status_string(0) == b"ok"
    assert lib.fbsr_version() >= 100
    assert lib.fbsr_stats_workspace_bytes() % 72 == 0


def test_argument_validation_needs_no_device(lib):
    vp, sz, i, u64, f = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_uint64, ctypes.c_float
    lib.fbsr_round.argtypes = [vp, vp, sz, i, i, i, u64, u64, f, vp]
    # invalid enum / k / scale are rejected before anything touches the device
    assert lib.fbsr_round(None, None, 0, 9, 0, 4, 0, 0, 1.0, None) == 1
    assert lib.fbsr_round(None, None, 0, 0, 6, 4, 0, 0, 1.0, None) == 1
    assert lib.fbsr_round(None, None, 0, 0, 0, 0, 0, 0, 1.0, None) == 1
    assert lib.fbsr_round(None, None, 0, 0, 0, 17, 0, 0, 1.0, None) == 1
    assert lib.fbsr_round(None, None, 0, 0, 0, 4, 0, 0, -1.0, None) == 1
    assert lib.fbsr_round(None, None, 8, 0, 0, 4, 0, 0, 1.0, None) == 1        # null pointers with n > 0
    assert lib.fbsr_round(2, 4, 8, 0, 0, 4, 0, 0, 1.0, None) == 3              # src not 4-byte aligned
    assert lib.fbsr_round(None, None, 0, 0, 0, 4, 0, 0, 1.0, None) == 0        # empty call is a no-op
    assert lib.fbsr_round(None, None, 0, 4, 0, 4, 0, 0, 1.0, None) == 0        # format 4 = Binary8P4
    assert lib.fbsr_round(None, None, 0, 5, 0, 4, 0, 0, 1.0, None) == 1


def test_binding_has_no_fallback():
    src = open(os.path.join(ROOT, "paper_2504_20634_b200", "binding.py")).read()
    assert "oracle" not in src
    for name in os.listdir(os.path.join(ROOT, "paper_2504_20634_b200")):
        if name.endswith(".py"):
            assert "import oracle" not in open(os.path.join(ROOT, "paper_2504_20634_b200", name)).read()
            assert "from oracle" not in open(os.path.join(ROOT, "paper_2504_20634_b200", name)).read()


def test_format_descriptor_validation(lib):
    """fbsr_format_desc_valid is host-only: the accepted ranges of the header, checked without a GPU."""
    import ctypes

    class Desc(ctypes.Structure):
        _fields_ = [("K", ctypes.c_int32), ("P", ctypes.c_int32), ("B", ctypes.c_int32), ("max_code", ctypes.c_uint32),
                    ("has_inf", ctypes.c_int32), ("inf_code", ctypes.c_uint32), ("nan_code", ctypes.c_uint32),
                    ("single_zero", ctypes.c_int32)]

    lib.fbsr_format_desc_valid.argtypes = [ctypes.POINTER(Desc)]
    ok = [(16, 8, 127, 0x7F7F, 1, 0x7F80, 0x7FC0, 0), (8, 4, 7, 0x7E, 0, 0, 0x7F, 0), (8, 4, 8, 0x7E, 1, 0x7F, 0x80, 1),
          (8, 3, 16, 0x7F, 0, 0, 0x80, 1), (16, 13, 4, 0x7FFE, 0, 0, 0x8000, 1)]
    bad = [(12, 4, 7, 0x7E, 0, 0, 0x7F, 0), (8, 1, 7, 0x7E, 0, 0, 0x7F, 0), (8, 8, 7, 0x7E, 0, 0, 0x7F, 0),
           (16, 14, 7, 0x7E, 0, 0, 0x7FFF, 0), (8, 4, 0, 0x7E, 0, 0, 0x7F, 0), (8, 4, 128, 0x7E, 0, 0, 0x7F, 0),
           (8, 4, 7, 0, 0, 0, 0x7F, 0), (8, 4, 7, 0x7E, 1, 0x7E, 0x7F, 0), (8, 4, 7, 0x7E, 1, 0x7F, 0x7F, 0),
           (8, 4, 7, 0x7E, 0, 0, 0x7D, 0), (8, 4, 7, 0x7E, 0, 0, 0x7F, 1), (16, 8, 100, 0x7F7F, 1, 0x7F80, 0x7FC0, 0)]
    for d in ok:
        assert lib.fbsr_format_desc_valid(ctypes.byref(Desc(*d))) == 1, d
    for d in bad:
        assert lib.fbsr_format_desc_valid(ctypes.byref(Desc(*d))) == 0, d
    assert lib.fbsr_format_desc_valid(None) == 0


def test_python_tile_table_equals_the_library(lib):
    """The shard grid of the host logic is built from a Python copy of the tile-size rule: it must be the
    library's for every draw width, and the shard alignment a multiple of each tile size."""
    import ctypes
    from paper_2504_20634_b200 import sharding
    lib.fbsr_tile_elements.argtypes = [ctypes.c_int]
    lib.fbsr_tile_elements.restype = ctypes.c_size_t
    for k in range(1, 17):
        assert sharding.tile_elements(k) == lib.fbsr_tile_elements(k), k
        assert sharding.SHARD_ALIGN % lib.fbsr_tile_elements(k) == 0
    assert lib.fbsr_tile_elements(0) == 0 and lib.fbsr_tile_elements(17) == 0


def test_adam_scalars_match_the_oracle_and_do_not_cost_the_step_count(lib):
    """The host scalars of the Adam steps equal the oracle's (which multiplies beta `step` times) bit for bit,
    including far into a run, where the library stops multiplying once beta^step can no longer matter."""
    import time
    import numpy as np
    from oracle import capi
    lib.fbsr_adam_scalars.argtypes = [ctypes.c_float, ctypes.c_float, ctypes.c_float, ctypes.c_int,
                                      ctypes.POINTER(ctypes.c_float)]
    lib.fbsr_adam_scalars.restype = None
    out = (ctypes.c_float * 4)()
    for lr, b1, b2 in ((1e-4, 0.9, 0.999), (3e-3, 0.5, 0.95), (1e-3, 0.0, 0.999), (1e-3, 0.99, 0.9999)):
        for step in (1, 2, 10, 353, 354, 5000, 37000, 38000, 400000, 10 ** 6):
            lib.fbsr_adam_scalars(lr, b1, b2, step, out)
            want = capi.adam_coefficients(lr, b1, b2, step)
            got = np.array(list(out), dtype=np.float32)
            assert np.array_equal(got.view(np.uint32), np.array(want, dtype=np.float32).view(np.uint32)), (lr, b1, b2, step)
    t0 = time.perf_counter()
    for _ in range(200):
        lib.fbsr_adam_scalars(1e-4, 0.9, 0.999, 2 ** 31 - 1, out)
    assert time.perf_counter() - t0 < 1.0                     # 200 x 2^31 multiplications would take minutes
