"""The C-ABI library builds, loads and exports every entry point the header declares.
No compute call is made here (this file runs without a GPU)."""
import ctypes
import os
import re

import pytest

from paper_2006_12608_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def declared_symbols():
    with open(os.path.join(ROOT, "include", "simjoin.h")) as f:
        text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    return sorted(set(re.findall(r"\b(simjoin_[a-z_0-9]+)\s*\(", text)))


def test_header_and_binding_agree():
    syms = declared_symbols()
    assert "simjoin_create" in syms and "simjoin_run" in syms and "simjoin_destroy" in syms
    assert sorted(binding.EXPORTS) == syms


def test_library_exports_every_declared_symbol(lib):
    for s in declared_symbols():
        assert hasattr(lib, s), s


def test_strerror_and_status_codes(lib):
    names = [binding.strerror(s) for s in range(7)]
    assert names[0] == "ok" and len(set(names)) == 7
    assert "unknown" in binding.strerror(99)


def test_argument_errors_need_no_gpu(lib):
    h = ctypes.c_void_p()
    assert lib.simjoin_create(None, 0, 0, None) == binding.SIMJOIN_ERR_ARG
    assert lib.simjoin_create(ctypes.byref(h), 7, 0, None) == binding.SIMJOIN_ERR_ARG
    cnt = ctypes.c_uint64(5)
    assert lib.simjoin_run(None, None, 0, None, 0, 16, 0, 0.0, None, 0, ctypes.byref(cnt)) == binding.SIMJOIN_ERR_ARG
    assert lib.simjoin_destroy(None) == binding.SIMJOIN_OK
    assert lib.simjoin_set_offsets(None, 0, 0) == binding.SIMJOIN_ERR_ARG
    assert lib.simjoin_last_kernel_ms(None, None, None) == binding.SIMJOIN_ERR_ARG


def test_create_without_usable_device_fails_cleanly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    h = ctypes.c_void_p()
    st = lib.simjoin_create(ctypes.byref(h), 0, 0, None)
    assert st in (binding.SIMJOIN_ERR_CUDA, binding.SIMJOIN_ERR_ARG) and not h.value


def test_product_path_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2006_12608_b200")
    for dirpath, _d, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                with open(os.path.join(dirpath, f)) as fh:
                    src = fh.read()
                assert not re.search(r"^\s*(from|import)\s+oracle|simjoin_oracle|liboracle|oracle/", src, flags=re.M), f


def test_argument_checks_that_need_no_gpu(lib):
    """Null handles and unknown enumerators are rejected before any CUDA call is made."""
    c = ctypes
    assert lib.simjoin_create(None, 0, 0, None) == binding.SIMJOIN_ERR_ARG
    assert lib.simjoin_set_option(None, binding.SIMJOIN_OPT_SELECT_MIN_OPS, 1.0) == binding.SIMJOIN_ERR_ARG
    assert lib.simjoin_set_offsets(None, 0, 0) == binding.SIMJOIN_ERR_ARG
    assert lib.simjoin_last_kernel_ms(None, None, None) == binding.SIMJOIN_ERR_ARG
    assert lib.simjoin_destroy(None) == binding.SIMJOIN_OK
    cnt = c.c_uint64(7)
    assert lib.simjoin_run(None, None, 0, None, 0, 16, 0, 0.0, None, 0, c.byref(cnt)) == binding.SIMJOIN_ERR_ARG
    assert lib.simjoin_run_noalloc(0, None, 5, None, 0, None, 0, 16, 0, 0.0, None, 0, c.byref(cnt)) == binding.SIMJOIN_ERR_ARG   # dtype
    assert lib.simjoin_run_noalloc(-1, None, 0, None, 0, None, 0, 16, 0, 0.0, None, 0, c.byref(cnt)) == binding.SIMJOIN_ERR_ARG  # device
