"""The C-ABI library builds, loads on a machine without a GPU and exports every entry point
that include/evln.h declares.  No compute call is made here."""
import ctypes
import os
import re

import pytest

from paper_2512_10310_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    B.build_library()
    return B.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "evln.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(evln[A-Z]\w*)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in evln.h but not exported"
    assert sorted(B.EXPORTS) == names


def test_struct_sizes_match_the_header_layout():
    # 9 ints + float + double after a size_t: no hidden padding surprises on LP64
    assert ctypes.sizeof(B.evlnStepParams) == 56
    assert ctypes.sizeof(B.evlnPagedParams) == 56
    assert ctypes.sizeof(B.evlnGatherParams) == 40


def test_error_strings(lib):
    assert B.error_string(B.EVLN_OK) == "EVLN_OK"
    assert B.error_string(B.EVLN_CACHE_FULL) == "EVLN_CACHE_FULL"
    assert B.error_string(99) == "EVLN_UNKNOWN_STATUS"


def test_create_without_gpu_fails_loudly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("this check is for machines without a GPU")
    with pytest.raises(B.EvlnError) as e:
        B.evlnCreate(0)
    assert e.value.status == B.EVLN_CUDA_ERROR


def test_null_handle_is_rejected(lib):
    p = B.step_params("bf16", 28, 4, 128, 0, 1, 8, 1e6)
    v = ctypes.c_size_t(0)
    assert lib.evlnStepWorkspaceSize(None, ctypes.byref(p), ctypes.byref(v)) == B.EVLN_INVALID_VALUE
    assert lib.evlnDestroy(None) == B.EVLN_INVALID_VALUE
