"""The C-ABI library loads on a machine without a GPU and exports what include/zipml.h declares."""
import ctypes as C
import os
import re

import pytest

import oracle
from paper_1611_05402_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1611_05402_b200.build import build
    build()
    return binding.lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "zipml.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(zipml_[a-z_0-9]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_host_only_helpers(lib):
    for bits in (1, 2, 3, 4, 5, 6, 7, 8):
        for n in (1, 7, 64, 1000, 2048, 32768):
            assert lib.zipml_row_bytes(n, bits) == oracle.row_bytes(n, bits)
    assert lib.zipml_row_bytes(10, 9) == 0 and lib.zipml_row_bytes(10, 0) == 0 and lib.zipml_row_bytes(0, 4) == 0
    assert lib.zipml_strerror(0) == b"ok"
    assert b"non-finite" in lib.zipml_strerror(binding.ERR_NONFINITE)
    assert C.sizeof(binding.CDataset) == 80 and C.sizeof(binding.CSgdParams) == 120


def test_no_device_is_an_error_not_a_fallback(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    h = C.c_void_p()
    assert lib.zipml_create(C.byref(h), 0, None) == binding.ERR_CUDA
    assert not h
    with pytest.raises(binding.ZipmlError):
        binding.Context("cuda:0")
    assert lib.zipml_sync(None) == binding.ERR_INVALID_ARG
    assert lib.zipml_destroy(None) == binding.OK


def test_product_code_never_touches_the_oracle():
    pkg = os.path.join(ROOT, "paper_1611_05402_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"import\s+oracle|from\s+oracle|liboracle|oracle/|oracle\.", text), f
