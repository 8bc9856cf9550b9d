"""CPU-only checks of the boundary: the library loads and exports every symbol
the header declares; host-side argument validation needs no GPU."""
import ctypes
import os
import re

import pytest

from paper_2405_16528_b200 import binding as L
from paper_2405_16528_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return L.lib()


def test_header_symbols_are_exported(lib):
    hdr = open(os.path.join(ROOT, "include", "loqt.h")).read()
    declared = set(re.findall(r"\b(loqt_[a-z0-9_]+)\s*\(", hdr))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared but not exported"
    assert declared == set(L.EXPORTS)


def test_status_strings(lib):
    assert lib.loqt_status_string(0) == b"ok"
    assert b"workspace" in lib.loqt_status_string(4)
    assert lib.loqt_status_string(99) == b"unknown status"


def test_workspace_sizes(lib):
    assert L.loqt_workspace_bytes(L.LOQT_OP_MERGE, 4096, 4096, 1024, 0) == 256 + 4096 * 1024 * 2
    fwd = L.loqt_workspace_bytes(L.LOQT_OP_FWD, 4096, 4096, 1024, 4096)
    assert fwd == 256 + 4096 * 1024 * 2
    assert L.loqt_workspace_bytes(L.LOQT_OP_BWD, 4096, 4096, 1024, 4096) >= fwd
    # r = 32 is padded to one 64-wide stage in the scratch matrix
    assert L.loqt_workspace_bytes(L.LOQT_OP_FWD, 256, 256, 32, 512) == 256 + 512 * 64 * 2


def test_host_validation_without_gpu(lib):
    bad = L.loqt_nf4_mat(None, None, 4, 64, 64, 64)
    assert lib.loqt_nf4_quantize(None, 64, bad, None) == 1          # null pointers
    m = L.loqt_nf4_mat(16, 16, 4, 64, 64, 32)
    assert lib.loqt_nf4_quantize(16, 64, m, None) == 3              # block size
    m = L.loqt_nf4_mat(16, 16, 4, 64, 96, 64)
    assert lib.loqt_nf4_quantize(16, 64, m, None) == 2              # ld not a multiple of 64
    assert lib.loqt_device_status(None, None) == 1
    assert lib.loqt_launch_count() == 0 or lib.loqt_launch_count() > 0


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(L, "_lib", None)
    monkeypatch.setattr(L, "LIB_PATH", "/nonexistent/libloqt.so")
    with pytest.raises(L.LoqtError, match="no CPU or PyTorch fallback"):
        L.lib()
