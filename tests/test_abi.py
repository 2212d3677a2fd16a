"""CPU-only checks of the boundary: the shared library builds, loads and exports every symbol the
header declares; argument errors are reported by status code before anything touches a GPU; and
without a GPU the product path fails loudly instead of falling back."""
import ctypes
import os
import re

import pytest
import torch

import paper_2503_24358_b200 as sq
from paper_2503_24358_b200 import build as sq_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    sq_build.build()
    return sq.binding._load()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "squat.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(squat_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(sq.EXPORTED_SYMBOLS)


def test_status_strings(lib):
    assert lib.squat_status_string(0) == b"ok"
    assert lib.squat_status_string(3) == b"configuration not built"
    assert lib.squat_status_string(99) == b"unknown status"


def test_argument_errors_come_back_as_status_codes(lib):
    h = ctypes.c_void_p()
    assert lib.squat_subspace_create(0, 128, ctypes.byref(h)) == 1          # invalid
    assert lib.squat_subspace_create(8, 64, ctypes.byref(h)) == 3           # head_dim not built
    assert lib.squat_subspace_create(8, 128, None) == 1
    # quantizers: NULL pointers, misaligned pointers, unsupported bits / group sizes
    z = ctypes.c_void_p(0)
    a = ctypes.c_void_p(4096)          # never dereferenced: validation fails first
    mis = ctypes.c_void_p(4100)
    assert lib.squat_quantize_values(z, 1, 1, 1, 32, 128, 0, 0, 128, 2, 32, a, a, a, 0, 0, None) == 1
    assert lib.squat_quantize_values(z, 1, 1, 1, 0, 128, 0, 0, 128, 2, 32, z, z, z, 0, 0, None) == 0      # empty: no-op
    assert lib.squat_quantize_values(mis, 1, 1, 1, 32, 128, 0, 0, 128, 2, 32, a, a, a, 0, 0, None) == 1
    assert lib.squat_quantize_values(a, 1, 1, 1, 32, 128, 0, 0, 128, 3, 32, a, a, a, 0, 0, None) == 3
    assert lib.squat_quantize_values(a, 1, 1, 1, 32, 128, 0, 0, 128, 2, 48, a, a, a, 0, 0, None) == 3
    assert lib.squat_quantize_values(a, 7, 1, 1, 32, 128, 0, 0, 128, 2, 32, a, a, a, 0, 0, None) == 1
    assert lib.squat_quantize_values(a, 1, 1, 1, 32, 128, 0, 0, 64, 2, 32, a, a, a, 0, 0, None) == 1   # stride_t < d
    assert lib.squat_quantize_values(a, 1, 1, 1, 32, 96, 0, 0, 96, 2, 64, a, a, a, 0, 0, None) == 2    # d % G
    assert lib.squat_quantize_keys(None, a, 1, 1, 1, 32, 128, 0, 0, 128, 2, 32, a, a, a, 0, 0, None) == 1
    assert lib.squat_dequantize(5, a, a, a, 1, 1, 32, 128, 2, 32, 0, 0, a, 0, None) == 1
    assert lib.squat_dequantize(0, a, a, a, 1, 1, 33, 128, 2, 32, 0, 0, a, 0, None) == 2               # T % G for keys
    assert lib.squat_dequantize(1, a, a, a, 1, 1, 33, 128, 8, 32, 0, 0, a, 0, None) == 3
    assert lib.squat_build_subspace_power(None, a, 0, 8, 32, 4096, 128, 8, 1e-3, 1, a, 0, 2, None) == 1
    assert lib.squat_build_subspace_power_from_gram(None, a, 8, 1e-3, 1, a, 0, 2, None) == 1
    assert lib.squat_get_device_status(None, None, 0) == 1
    assert lib.squat_write_path_workspace_bytes(1, 1, 32, 32, 4096, 128, 2, 32) > 2 * 32 * 4096 * 128 * 2


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks behaviour on a machine without a GPU")
def test_no_gpu_means_loud_failure_not_fallback(lib):
    with pytest.raises(sq.SquatError):
        sq.Subspace(8, 128)
    with pytest.raises(ValueError):
        sq.squat_quantize_values(torch.zeros(1, 1, 32, 128), 2, 32, torch.zeros(1), torch.zeros(1), torch.zeros(1))


def test_package_does_not_import_the_oracle():
    import sys
    pkg_dir = os.path.join(ROOT, "paper_2503_24358_b200")
    for dirpath, _, files in os.walk(pkg_dir):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src and "squat_oracle" not in src, f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c", ".h")):
            assert "paper_2503_24358_b200" not in open(os.path.join(ROOT, "oracle", f)).read(), f


def test_rope_table_is_cos_sin_of_block_and_lane_angles():
    # host-side function of the library (no GPU): (cos, sin) of 32 a theta_i for every block a of 32 positions, then of
    # l theta_i for l < 32, theta_i = base^(-2 i / 128) -- checked against math.cos / math.sin
    import math
    import paper_2503_24358_b200 as sq
    for base, npos in ((10000.0, 100), (500000.0, 33)):
        t = sq.squat_rope_table(npos, base).numpy().reshape(-1, 64, 2)
        nb = (npos + 31) // 32
        assert t.shape[0] == nb + 32
        for row, pos in [(a, 32 * a) for a in range(nb)] + [(nb + l, l) for l in range(32)]:
            for i in (0, 1, 31, 63):
                ang = pos * base ** (-2.0 * i / 128)
                assert abs(t[row, i, 0] - math.cos(ang)) <= 6e-8 and abs(t[row, i, 1] - math.sin(ang)) <= 6e-8
