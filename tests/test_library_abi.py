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


def test_struct_sizes_match_the_header_layout(tmp_path):
    # what the C compiler makes of include/evln.h is what the ctypes structures must be
    import subprocess
    src = tmp_path / "sizes.c"
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "evln.h"\n'
                   'int main(void) { printf("%zu %zu %zu %zu %zu\\n", sizeof(evlnStepParams), sizeof(evlnPagedParams), '
                   'sizeof(evlnGatherParams), offsetof(evlnStepParams, rope_table), offsetof(evlnGatherParams, rope_table)); '
                   'printf("%zu\\n", offsetof(evlnPagedParams, rope_table)); '
                   'return 0; }\n')
    exe = tmp_path / "sizes"
    subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)])
    step, paged, gather, off_step, off_gather, off_paged = map(int, subprocess.check_output([str(exe)]).split())
    assert ctypes.sizeof(B.evlnStepParams) == step == 72
    assert ctypes.sizeof(B.evlnPagedParams) == paged == 72
    assert ctypes.sizeof(B.evlnGatherParams) == gather == 56
    assert B.evlnStepParams.rope_table.offset == off_step
    assert B.evlnGatherParams.rope_table.offset == off_gather
    assert B.evlnPagedParams.rope_table.offset == off_paged


def test_page_table_check_on_the_host(lib):
    # no GPU involved: range, duplicates within and across episodes, short tables
    p = B.paged_params(28, 4, 128, 2, 64, 16, 8, 1e6)
    ok = [[0, 1, 9, 9, 9, 9, 9, 9], [2, 3, 9, 9, 9, 9, 9, 9]]           # entries past the needed pages are ignored
    assert B.evlnPagedCheckTable(p, [100, 70], [0, 10, 20], ok) == (B.EVLN_OK, -1, -1)
    assert B.evlnPagedCheckTable(p, [100, 70], [0, 10, 20], [[0, 1] + [9] * 6, [2, 1] + [9] * 6]) == (B.EVLN_INVALID_VALUE, 1, 1)
    assert B.evlnPagedCheckTable(p, [100, 70], [0, 10, 20], [[0, 0] + [9] * 6, [2, 3] + [9] * 6]) == (B.EVLN_INVALID_VALUE, 0, 1)
    assert B.evlnPagedCheckTable(p, [100, 70], [0, 10, 20], [[0, 16] + [9] * 6, [2, 3] + [9] * 6]) == (B.EVLN_INVALID_VALUE, 0, 1)
    assert B.evlnPagedCheckTable(p, [100, 70], [0, 10, 20], [[0, -1] + [9] * 6, [2, 3] + [9] * 6]) == (B.EVLN_INVALID_VALUE, 0, 1)
    assert B.evlnPagedCheckTable(p, [600, 70], [0, 10, 20], ok)[0] == B.EVLN_CACHE_FULL      # 10 pages needed, 8 per row
    assert B.evlnRopeTableBytes(128, 196) == 196 * 64 * 16 and B.evlnRopeTableBytes(96, 4) == 0


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
