"""The C-ABI library builds, loads and exports every entry point the header declares (no GPU needed)."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1909_04885_b200 import build, binding
    build.build()
    return binding.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "chicle.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(chicle_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_1909_04885_b200 import binding
    names = declared_functions()
    assert len(names) >= 12
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTED) == [n for n in names if n in binding.EXPORTED]
    assert set(names) == set(binding.EXPORTED)


def test_null_and_argument_errors_need_no_gpu(lib):
    from paper_1909_04885_b200 import binding
    assert lib.chicle_partition(None, 4, 0) == 1
    assert lib.chicle_cocoa_round(None, 0, 1.0, None) == 1
    assert lib.chicle_duality_gap(None, None, None, None) == 1
    lib.chicle_glm_destroy(None)
    h = ctypes.c_void_p()
    vals = np.ones(4, np.float32)
    y = np.ones(2, np.float32)
    m = binding.Matrix(0, 0, 2, 2, 0, 2, None, None, vals.ctypes.data_as(ctypes.c_void_p))
    yp = y.ctypes.data_as(ctypes.c_void_p)
    assert lib.chicle_glm_create(ctypes.byref(m), yp, ctypes.c_float(-1.0), 0, 0, None, None, ctypes.byref(h)) == 1
    assert b"lambda" in lib.chicle_last_error(None)
    m2 = binding.Matrix(0, 0, 2, 2, 0, 2, None, None, vals.ctypes.data_as(ctypes.c_void_p))
    assert lib.chicle_glm_create(ctypes.byref(m2), yp, ctypes.c_float(1.0), 2, 0, None, None, ctypes.byref(h)) == 5
    assert h.value is None


def test_create_without_a_gpu_fails_loudly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_1909_04885_b200 import binding
    with pytest.raises(binding.ChicleError) as ei:
        binding.Glm("hinge", "dense", 2, 2, np.ones(4, np.float32), np.ones(2, np.float32), 0.1,
                    torch_allocator=False, stream=0)
    assert ei.value.status == 4 and "no host path" in str(ei.value)


def test_errors_are_logged_when_asked(lib):
    # CHICLE_LOG=1: a failed call writes a line to stderr (the variable is read once, so in a process of its own)
    import subprocess
    import sys
    code = ("import ctypes, numpy as np\n"
            "from paper_1909_04885_b200 import binding\n"
            "lib = binding.load()\n"
            "h = ctypes.c_void_p(); vals = np.ones(4, np.float32); y = np.ones(2, np.float32)\n"
            "m = binding.Matrix(0, 0, 2, 2, 0, 2, None, None, vals.ctypes.data_as(ctypes.c_void_p))\n"
            "st = lib.chicle_glm_create(ctypes.byref(m), y.ctypes.data_as(ctypes.c_void_p), ctypes.c_float(-1.0), 0, 0, None, None, ctypes.byref(h))\n"
            "assert st == 1\n")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    for level, expect in (("1", True), ("0", False)):
        env = dict(os.environ, CHICLE_LOG=level, PYTHONPATH=root)
        r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=300)
        assert r.returncode == 0, r.stderr
        assert ("[chicle] error 1" in r.stderr and "lambda" in r.stderr) == expect
