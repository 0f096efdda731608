"""Host-side checks that need no GPU: the shared library builds, loads, exports every symbol the
header declares, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2512_09963_b200 import binding as B
from paper_2512_09963_b200 import build as gs_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "goodspeed.h")


@pytest.fixture(scope="module")
def lib():
    gs_build.build()
    return B.lib()


def declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gs_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = declared_symbols()
    assert "gs_verify_attn" in names and "gs_lm_head_logits" in names
    assert "gs_spec_accept" in names and "gs_schedule" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in goodspeed.h but not exported"
        assert n in B.SIGNATURES, f"{n} has no ctypes signature"
        assert hasattr(B, n), f"{n} has no Python binding of the same name"


def test_status_strings_and_version(lib):
    assert B.gs_version() >= 100
    assert B.gs_status_str(0) == "ok"
    assert "workspace" in B.gs_status_str(4)


def test_argument_errors_are_synchronous(lib):
    null = None
    # negative sizes / null pointers: rejected before any CUDA call
    assert lib.gs_schedule(null, null, -1, 4, null, null, null, null, null) == 1
    assert lib.gs_schedule(null, null, 4, 4, null, null, null, null, null) == 1
    assert lib.gs_schedule(null, null, 0, 4, null, null, null, null, null) == 0       # empty: nothing to do
    assert lib.gs_schedule(ctypes.c_void_p(8), ctypes.c_void_p(8), 5000, 4, null, null, ctypes.c_void_p(8),
                           null, null) == 3
    assert lib.gs_spec_accept(null, null, null, null, null, null, 1.0, 4, 2, 100, null, null, null, null,
                              null, null, null, null, 0.1, 0.5, 0.0, 1.0, null, 0, null, null) == 2  # Tq < N
    assert lib.gs_spec_accept(null, null, null, null, null, null, -1.0, 4, 8, 100, null, null, null, null,
                              null, null, null, null, 0.1, 0.5, 0.0, 1.0, null, 0, null, null) == 1  # tau < 0
    assert lib.gs_spec_accept(null, null, null, null, null, null, 1.0, 0, 0, 100, null, null, null, null,
                              null, null, null, null, 0.1, 0.5, 0.0, 1.0, null, 0, null, null) == 0  # N = 0
    assert lib.gs_lm_head_logits(null, null, null, 4, 8, 8, 1, null, 0, null, null) == 1
    assert lib.gs_lm_head_logits(null, null, null, 0, 8, 8, 1, null, 0, null, null) == 0
    assert lib.gs_lm_head_logits(null, null, null, 4, 8, 8, 7, null, 0, null, null) == 1             # dtype
    assert lib.gs_verify_attn(null, null, null, null, null, null, 2, 4, 10, 10, 8, 3, 64, 0.125, 1,
                              null, 0, null, null) == 1
    p = ctypes.c_void_p(256)
    assert lib.gs_verify_attn(p, p, p, p, p, p, 2, 4, 10, 10, 8, 3, 64, 0.125, 1, p, 1 << 20, null, null) == 2
    assert lib.gs_verify_attn(p, p, p, p, p, p, 2, 4, 10, 10, 8, 4, 64, 0.125, 1, null, 0, null, null) == 4


def test_workspace_queries(lib):
    # at least one (max, argmax, sum) statistic per row and chunk of 8192 columns
    assert B.gs_spec_accept_workspace(8, 44, 151936) >= 44 * ((151936 + 8191) // 8192) * 12
    assert B.gs_spec_accept_workspace(8, 44, 151936) % 256 == 0
    assert B.gs_lm_head_workspace(44, 5120, 151936, B.GS_BF16) >= 0
    assert B.gs_verify_attn_workspace(8, 44, 16424, 2053, 64, 8, 128, B.GS_BF16) >= 0


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="missing"):
        B.lib()
