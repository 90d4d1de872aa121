"""The C-ABI library loads without a GPU and exports every function include/hq.h declares."""
from __future__ import annotations

import ctypes
import os
import re

import pytest

from paper_2011_10680_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libhq():
    build.build()
    return ctypes.CDLL(build.LIB)


def declared_functions():
    text = open(os.path.join(ROOT, "include", "hq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hq_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_five_named_entry_points():
    names = declared_functions()
    for must in ("hq_conv2d", "hq_linear", "hq_residual_add", "hq_avgpool_requant", "hq_run_network"):
        assert must in names


def test_every_declared_function_is_exported(libhq):
    for name in declared_functions():
        assert hasattr(libhq, name), f"{name} declared in hq.h but not exported"
    assert set(binding.EXPORTS) <= set(declared_functions())


def test_status_strings_and_loud_failure_without_gpu(libhq):
    libhq.hq_status_string.restype = ctypes.c_char_p
    assert libhq.hq_status_string(0) == b"HQ_OK"
    assert libhq.hq_status_string(7) == b"HQ_ERR_TIMEOUT"
    import torch
    if not torch.cuda.is_available():
        h = ctypes.c_void_p()
        assert libhq.hq_create(0, ctypes.byref(h)) != 0      # no CPU fallback: creation fails
        assert not h.value


def test_struct_layouts_match_the_header():
    # sizes implied by the field lists of hq.h on an LP64 machine
    assert ctypes.sizeof(binding.hq_tensor) == 32
    assert ctypes.sizeof(binding.hq_dyadic) == 16
    assert ctypes.sizeof(binding.hq_conv_desc) == 104
    assert ctypes.sizeof(binding.hq_layer) == 352


def test_cuda_sources_have_no_floating_point():
    csrc = os.path.join(ROOT, "paper_2011_10680_b200", "csrc")
    for f in os.listdir(csrc):
        if "__global__" not in open(os.path.join(csrc, f)).read():
            continue                      # host-only files (API glue, event timing) are not the pipeline
        code = re.sub(r"//[^\n]*", "", open(os.path.join(csrc, f)).read())
        code = re.sub(r"/\*.*?\*/", "", code, flags=re.S)
        assert not re.search(r"\b(float|double|__half|half2|__nv_bfloat16)\b", code), f
