"""The C boundary: the library builds, loads without a GPU and exports what the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libs():
    from paper_1906_12043_b200 import build
    return build.build()


def declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in sorted(os.listdir(inc)):
        src = open(os.path.join(inc, f)).read()
        src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
        names |= set(re.findall(r"\b(cocod_[a-z_0-9]+)\s*\(", src))
    return sorted(names)


def test_header_declares_the_five_calls_of_the_algorithm():
    names = declared_functions()
    for n in ("cocod_create", "cocod_local_step", "cocod_comm_begin", "cocod_comm_end", "cocod_destroy"):
        assert n in names


def test_library_exports_every_declared_symbol(libs):
    lib = ctypes.CDLL([p for p in libs if p.endswith("libcocod.so")][0])
    for n in declared_functions():
        assert hasattr(lib, n), f"{n} is declared in cocod.h but not exported"


def test_binding_covers_every_declared_symbol(libs):
    from paper_1906_12043_b200 import engine, mlp
    assert sorted(list(engine.SIGNATURES) + list(mlp.SIGNATURES)) == declared_functions()
    engine.load()
    mlp.load()


def test_error_paths_that_touch_no_device(libs):
    from paper_1906_12043_b200 import engine
    lib = engine.load()
    assert lib.cocod_strerror(0) == b"ok"
    for code in (-1, -2, -3, -4, -5):
        assert lib.cocod_strerror(code) not in (b"ok", b"unknown error code")
    assert lib.cocod_strerror(-99) == b"unknown error code"
    assert lib.cocod_local_step(None, None) == engine.ERR_INVALID
    assert lib.cocod_comm_begin(None, None) == engine.ERR_INVALID
    assert lib.cocod_comm_end(None) == engine.ERR_INVALID
    assert lib.cocod_destroy(None) == engine.OK
    out = ctypes.c_void_p()
    assert lib.cocod_create(ctypes.byref(out), 0, 10, 0.1, 0.9, 0.0) == engine.ERR_INVALID
    assert lib.cocod_create(ctypes.byref(out), 4, 0, 0.1, 0.9, 0.0) == engine.ERR_INVALID
    assert lib.cocod_create(ctypes.byref(out), 4, 10, float("nan"), 0.9, 0.0) == engine.ERR_INVALID
    assert lib.cocod_create(ctypes.byref(out), 1024, 2 ** 61, 0.1, 0.9, 0.0) == engine.ERR_INVALID
    assert lib.cocod_create(None, 4, 10, 0.1, 0.9, 0.0) == engine.ERR_INVALID
    assert lib.cocod_kernel_mean(None, 4, 10, None, None, None) == engine.ERR_INVALID
    from paper_1906_12043_b200 import mlp
    mlp.load()
    assert lib.cocod_mlp_create(None, 2, 128, 784, 1024, 10) == engine.ERR_INVALID
    assert lib.cocod_mlp_create(ctypes.byref(out), 2, 64, 784, 1024, 10) == engine.ERR_INVALID
    assert lib.cocod_mlp_create(ctypes.byref(out), 2, 128, 783, 1024, 10) == engine.ERR_INVALID
    assert lib.cocod_mlp_create(ctypes.byref(out), 2, 128, 784, 1000, 10) == engine.ERR_INVALID
    assert lib.cocod_mlp_create(ctypes.byref(out), 2, 128, 784, 1024, 17) == engine.ERR_INVALID
    assert lib.cocod_mlp_grad(None, None, None, None, None, None, None) == engine.ERR_INVALID
    assert lib.cocod_mlp_destroy(None) == engine.OK
    assert lib.cocod_gemm_bf16(None, None, None, 1, 1, 1, 1, 0, 0, 8, 8, 8, 8, 8, 8, None) == engine.ERR_INVALID


def test_engine_refuses_to_run_without_a_gpu(libs):
    import torch
    from paper_1906_12043_b200 import engine
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError):
        engine.Engine(2, 8, 0.1, 0.9, 0.0)


def test_inputs_library_exports_its_generators(libs):
    lib = ctypes.CDLL([p for p in libs if p.endswith("libcocod_inputs.so")][0])
    assert hasattr(lib, "cocod_inputs_gaussian_f32") and hasattr(lib, "cocod_inputs_gaussian_bf16")
