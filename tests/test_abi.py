"""The C-ABI library loads and exports what include/pw.h declares; host-only calls behave (CPU only)."""
import ctypes as C
import os
import re

import pytest

from paper_2607_16184_b200 import binding as B
from paper_2607_16184_b200 import build as pwbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    pwbuild.build()
    return B.load()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "pw.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(pw_[a-z_]+)\s*\(", header))
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_page_bytes_matches_size_table(lib, orc):
    for rows, cols in ((128, 128), (14336, 4096), (4096, 14336), (1408, 2048)):
        for bits in (16, 8, 4, 3, 2):
            assert B.pw_page_bytes(rows, cols, bits) == orc.page_bytes(rows, cols, bits)
    assert B.pw_page_bytes(128, 100, 4)[0] == 0
    assert B.pw_page_bytes(128, 128, 5)[0] == 0
    assert B.pw_page_bytes(128, 128, 4, group=64)[0] == 0


def test_status_strings_and_null_arguments(lib):
    assert lib.pw_status_str(0) == b"ok"
    assert b"timed out" in lib.pw_status_str(8)
    assert lib.pw_create(None, None) == 1
    assert lib.pw_workspace_bytes(None) == 0
    cfg = B.pw_config(1, 8, 0, 256, 512, 128, 16, 2, None, 0)
    assert lib.pw_workspace_bytes(C.byref(cfg)) > 0
    bad = B.pw_config(1, 8, 0, 250, 512, 128, 16, 2, None, 0)
    assert lib.pw_workspace_bytes(C.byref(bad)) == 0
    h = C.c_void_p()
    assert lib.pw_create(C.byref(h), C.byref(bad)) == 2          # PW_ERR_SHAPE, nothing touched
    assert lib.pw_create(C.byref(h), C.byref(cfg)) == 1          # no workspace given
    assert lib.pw_destroy(None) == 1
    assert lib.pw_launch_count(None) == 0


def test_workspace_grows_with_the_configuration(lib):
    small = B.pw_config(1, 8, 0, 256, 512, 128, 16, 2, None, 0)
    big = B.pw_config(32, 8, 0, 4096, 14336, 128, 64, 2, None, 0)
    assert lib.pw_workspace_bytes(C.byref(big)) > lib.pw_workspace_bytes(C.byref(small))
