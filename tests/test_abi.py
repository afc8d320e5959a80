"""The C-ABI library: it builds, loads, exports every symbol include/anpd.h declares, and
refuses to work without a CUDA device instead of computing anything on the CPU."""
import os
import re

import numpy as np
import pytest
import torch

from paper_2404_08698_b200 import binding as A, build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    B.build()
    return A.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "anpd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(anpd_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = declared_functions()
    assert "anpd_ngram_update" in names and "anpd_ngram_draft" in names
    assert "anpd_verify" in names and "anpd_generate" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(A.SIGNATURES) == names


def test_status_strings(lib):
    assert A.status_string(0) == "ok"
    assert "range" in A.status_string(A.ERR_RANGE)


def test_argument_errors_need_no_gpu(lib):
    cfg = A.NgramConfig(1, 3, 64, 0)           # n_min < 2
    out = A._P()
    assert lib.anpd_ngram_create(A.C.byref(cfg), None, A.C.byref(out)) == A.ERR_RANGE
    cfg = A.NgramConfig(2, 9, 64, 0)           # n_max > ANPD_N_MAX
    assert lib.anpd_ngram_create(A.C.byref(cfg), None, A.C.byref(out)) == A.ERR_RANGE
    assert lib.anpd_ngram_create(None, None, A.C.byref(out)) == A.ERR_ARG
    assert lib.anpd_model_destroy(None) == A.ERR_ARG
    assert lib.anpd_kv_truncate(None, 0, 0) == A.ERR_ARG


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device behaviour")
def test_no_cpu_fallback_without_a_device(lib):
    with pytest.raises(A.AnpdError) as e:
        A.anpd_ngram_create(2, 3, 64)
    assert e.value.status == A.ERR_CUDA
    from workloads import ModelShape, make_weights, tensor_shapes
    shape = ModelShape(1, 64, 1, 1, 64, 64, 32)
    w = make_weights(shape, 0, False)
    with pytest.raises(A.AnpdError) as e:
        A.anpd_model_create(shape, [w[n] for n, _ in tensor_shapes(shape)])
    assert e.value.status == A.ERR_CUDA


def test_product_code_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2404_08698_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src, f
    for dirpath, _, files in os.walk(os.path.join(ROOT, "oracle")):
        for f in files:
            if f.endswith(".py"):
                src = open(os.path.join(dirpath, f)).read()
                assert "paper_2404_08698_b200" not in src and "ctypes" not in src, f
