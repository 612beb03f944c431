"""Host-side checks of the C-ABI library that need no GPU: it loads, exports what the header declares,
rejects bad arguments before touching the device, and reproduces the generator's known answers."""
import ctypes
import os
import re

import pytest

import paper_2511_16652_b200 as egr
from paper_2511_16652_b200 import api

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _built():
    from paper_2511_16652_b200 import build
    build.build()
    return egr.load_library()


def test_library_exports_every_declared_symbol():
    lib = _built()
    header = "".join(open(os.path.join(ROOT, "include", h)).read() for h in sorted(os.listdir(os.path.join(ROOT, "include"))))
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(egr_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(api.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_version_and_error_strings():
    _built()
    assert egr.egr_version() >= 100
    assert egr.egr_strerror(0) == "ok"
    for code in range(-6, 0):
        assert "unknown" not in egr.egr_strerror(code)


def test_host_philox_known_answers():
    _built()
    path = os.path.join(ROOT, "tests", "golden", "philox4x32_10_kat.txt")
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        v = [int(t, 16) for t in line.split()]
        assert egr.egr_philox4x32_10(v[0:4], v[4:6]) == v[6:10]


def test_bad_arguments_are_rejected_before_any_device_work():
    lib = _built()
    L = egr.Layer(64, 64, 32, rank=3)                       # rank not a power of two <= 16
    fake = ctypes.c_void_p(4096)
    rc = lib.egr_perturbed_linear(ctypes.byref(L.c), fake, fake, ctypes.c_float(0.1), fake, fake, 1 << 20, None)
    assert rc == -1
    L = egr.Layer(64, 64, 31, rank=1, flags=egr.ANTITHETIC)  # odd population with pairs
    rc = lib.egr_perturbed_linear(ctypes.byref(L.c), fake, fake, ctypes.c_float(0.1), fake, fake, 1 << 20, None)
    assert rc == -1
    L = egr.Layer(64, 64, 32, rank=1, ldx=60)                # pitch smaller than the row
    rc = lib.egr_perturbed_linear(ctypes.byref(L.c), fake, fake, ctypes.c_float(0.1), fake, fake, 1 << 20, None)
    assert rc == -1
    L = egr.Layer(64, 64, 32, rank=1, ldx=68)                # bf16 pitch not a multiple of 8
    rc = lib.egr_perturbed_linear(ctypes.byref(L.c), fake, fake, ctypes.c_float(0.1), fake, fake, 1 << 20, None)
    assert rc == -2
    L = egr.Layer(64, 64, 32, rank=1)
    rc = lib.egr_perturbed_linear(ctypes.byref(L.c), ctypes.c_void_p(4098), fake, ctypes.c_float(0.1), fake, fake,
                                  1 << 20, None)
    assert rc == -2                                           # misaligned X
    rc = lib.egr_perturbed_linear(ctypes.byref(L.c), fake, fake, ctypes.c_float(0.1), fake, fake, 16, None)
    assert rc == -4                                           # workspace too small
    L = egr.Layer(64, 64, 32, rank=1, x_dtype=egr.F32)        # mixed dtypes
    rc = lib.egr_perturbed_linear(ctypes.byref(L.c), fake, fake, ctypes.c_float(0.1), fake, fake, 1 << 20, None)
    assert rc == -3
    L = egr.Layer(64, 64, 1 << 30, 2, 1)                      # 2^31 rows: beyond the kernel's 32-bit row coordinates
    rc = lib.egr_perturbed_linear(ctypes.byref(L.c), fake, fake, ctypes.c_float(0.1), fake, fake, 1 << 40, None)
    assert rc == -3
    rc = lib.egr_fitness_shape(fake, 0, 1, ctypes.c_void_p(8192), fake, 1 << 20, None)
    assert rc == -1
    rc = lib.egr_fitness_shape(fake, 8, 7, ctypes.c_void_p(8192), fake, 1 << 20, None)
    assert rc == -1
    Li = egr.Layer(64, 64, 32, rank=4, x_dtype=egr.I8, w_dtype=egr.I8, y_dtype=egr.I8)
    rc = lib.egr_perturbed_linear_i8(ctypes.byref(Li.c), fake, fake, 8, 7, fake, 20, fake, fake, 1 << 20, None)
    assert rc == -1                                           # integer path is rank 1 only


def test_no_cpu_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    lib = _built()
    fake = ctypes.c_void_p(4096)
    L = egr.Layer(64, 64, 32, rank=1)
    rc = lib.egr_perturbed_linear(ctypes.byref(L.c), fake, fake, ctypes.c_float(0.1), fake, fake, 1 << 20, None)
    assert rc == -5
    rc = lib.egr_fitness_shape(fake, 8, 1, ctypes.c_void_p(8192), fake, 1 << 20, None)
    assert rc == -5


def test_workspace_sizes():
    _built()
    L = egr.Layer(4096, 4096, 1024, rank=4)
    assert egr.egr_workspace_bytes(L, egr.OP_PERTURBED_LINEAR) >= 256 + 1024 * 4 * 4
    assert egr.egr_workspace_bytes(L, egr.OP_ES_UPDATE) >= 256 + 2 * 4096 * 4096 * 2
    assert egr.egr_workspace_bytes(egr.Layer(1, 1, 1000), egr.OP_FITNESS_SHAPE) >= 256 + 2 * 1000 * 8 + 2 * 256 * 4
