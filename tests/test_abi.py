"""The C-ABI library loads without a GPU and exports every symbol include/qarl.h declares."""
import ctypes
import os
import re

import pytest

from paper_2604_07853_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def test_exports_match_header(lib):
    header = open(os.path.join(ROOT, "include", "qarl.h")).read()
    code = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(qarl_[a-z_0-9]+)\s*\(", code))
    assert declared == set(binding.EXPORTS)
    hdr2 = re.sub(r"/\*.*?\*/", "", open(os.path.join(ROOT, "include", "qarl_harness.h")).read(), flags=re.S)
    declared2 = set(re.findall(r"\b(qarl_[a-z_0-9]+)\s*\(", hdr2))
    assert declared2 == set(binding.HARNESS_EXPORTS)
    for name in declared | declared2:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    for code in range(0, -9, -1):
        s = lib.qarl_status_string(code)
        assert s and s != b"unknown status"
    assert lib.qarl_status_string(-99) == b"unknown status"


def test_workspace_queries_are_host_only(lib):
    assert lib.qarl_linear_workspace_bytes(0, 256, 512) == 0
    n = lib.qarl_linear_workspace_bytes(16, 256, 512)
    assert n >= 16 * 512 + 16 * 4 * 4 and n % 256 == 0
    assert lib.qarl_moe_workspace_bytes(0, 2048, 768, 128, 8) == 0
    small = lib.qarl_moe_workspace_bytes(256, 2048, 768, 128, 8)
    big = lib.qarl_moe_workspace_bytes(512, 2048, 768, 128, 8)
    P = 256 * 8
    assert small >= P * 2048 + P * 768 + P * 2048 * 2 and big > small and small % 256 == 0


def test_create_fails_loudly_without_device(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    h = ctypes.c_void_p()
    rc = lib.qarl_create(ctypes.byref(h), 0)
    assert rc == -5 and not h.value
    with pytest.raises(binding.QarlError):
        binding.Context(0)


def test_no_oracle_in_product_path():
    """The package must not import, link or read anything under oracle/."""
    pkg = os.path.join(ROOT, "paper_2604_07853_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                bad = re.search(r"^\s*(import|from)\s+oracle|oracle[/.]|libqarl_oracle|#include.*oracle",
                                text, flags=re.M)
                assert bad is None, (os.path.join(dirpath, f), bad.group(0))
