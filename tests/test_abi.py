"""Host-side checks of the C ABI that need no GPU: the library loads, exports every
function the header declares, and rejects bad arguments before enqueuing anything."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2204_00595_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    entry.build()
    return B.lib()


def _declared():
    names = []
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b(monarch_\w+)\s*\(", text)
    return sorted(set(names))


def test_every_declared_symbol_is_exported(lib):
    declared = _declared()
    assert len(declared) >= 11
    for name in declared:
        assert hasattr(lib, name), name
    assert set(B.exported_symbols()) == set(declared)


def test_status_strings(lib):
    assert B.monarch_status_string(0) == "ok"
    seen = {B.monarch_status_string(s) for s in range(6)}
    assert len(seen) == 6


def test_workspace_bytes(lib):
    assert B.monarch_workspace_bytes(B.OP_FWD, 64, 256, 16, B.F32) >= 256
    assert B.monarch_workspace_bytes(B.OP_FWD, 64, 255, 16, B.F32) == 0      # n != m*m
    assert B.monarch_workspace_bytes(B.OP_FWD, 64, 9, 3, B.F32) == 0         # m not built
    assert B.monarch_workspace_bytes(7, 64, 256, 16, B.F32) == 0             # bad op
    assert B.monarch_workspace_bytes(B.OP_FWD, -1, 256, 16, B.F32) == 0


def test_argument_errors_return_before_launch(lib):
    f = lib.monarch_fwd
    ok_ptr = 0x10000                     # never dereferenced: every call below must fail first
    ws = 0x900000
    big = 1 << 30
    # n != m*m
    assert f(ok_ptr, ok_ptr + 4096, ok_ptr + 8192, ok_ptr + 12288, 1, 250, 16, 0, ws, big, None) == 1
    # unsupported m
    assert f(ok_ptr, ok_ptr, ok_ptr, ok_ptr, 1, 9, 3, 0, ws, big, None) == 2
    # bad dtype
    assert f(ok_ptr, ok_ptr, ok_ptr, ok_ptr, 1, 256, 16, 5, ws, big, None) == 1
    # null pointer
    assert f(None, 0x20000, 0x30000, 0x40000, 1, 256, 16, 0, ws, big, None) == 1
    # misaligned pointer
    assert f(0x10004, 0x20000, 0x30000, 0x40000, 1, 256, 16, 0, ws, big, None) == 1
    # output overlaps input
    assert f(0x10000, 0x20000, 0x30000, 0x10100, 1, 256, 16, 0, ws, big, None) == 1
    # workspace: missing, misaligned, too small
    assert f(0x10000, 0x20000, 0x30000, 0x40000, 1, 256, 16, 0, None, big, None) == 3
    assert f(0x10000, 0x20000, 0x30000, 0x40000, 1, 256, 16, 0, ws + 16, big, None) == 3
    assert f(0x10000, 0x20000, 0x30000, 0x40000, 1, 256, 16, 0, ws, 16, None) == 3
    # negative token count
    assert f(0x10000, 0x20000, 0x30000, 0x40000, -1, 256, 16, 0, ws, big, None) == 1
    g = lib.monarch_bwd_dw
    assert g(0x10000, 0x20000, 0x30000, 0x40000, 0x50000, 0x60000, 2, 1, 256, 16, 0, ws, big, None) == 1
    assert g(0x10000, 0x20000, 0x30000, 0x40000, 0x50000, 0x50000, 0, 1, 256, 16, 0, ws, big, None) == 1


def test_impl_selection(lib):
    prev = B.monarch_set_impl(B.IMPL_STAGED)
    try:
        assert B.monarch_impl_name(B.OP_FWD, 16, B.F32) == "staged-simt"
        assert B.monarch_set_impl(99) == -1
        assert B.monarch_impl_name(B.OP_FWD, 3, B.F32) == "unsupported"
    finally:
        B.monarch_set_impl(prev)


def test_deterministic_switch_changes_only_the_split_token_backward_workspaces(lib):
    """monarch_set_deterministic: returns the previous setting; while on, the workspace of the bf16 m = 32 and m = 64
    calls that sum weight gradients over token slices grows by the 32 MiB of partial sums; every other query
    (fp32, m = 128, forward, dx) is unchanged."""
    T = 1000
    def sizes():
        return {(op, m, dt): B.monarch_workspace_bytes(op, T, m * m, m, dt)
                for op in (B.OP_FWD, B.OP_BWD_DX, B.OP_BWD_DW, B.OP_BWD, B.OP_MLP_FWD)
                for m, dt in ((16, B.F32), (32, B.BF16), (64, B.BF16), (64, B.F32), (128, B.BF16))}
    before = sizes()
    assert B.monarch_set_deterministic(True) is False
    try:
        assert B.monarch_set_deterministic(True) is True
        after = sizes()
    finally:
        B.monarch_set_deterministic(False)
    grown = {k for k in before if after[k] != before[k]}
    assert grown == {(B.OP_BWD_DW, 64, B.BF16), (B.OP_BWD, 64, B.BF16), (B.OP_BWD_DW, 32, B.BF16), (B.OP_BWD, 32, B.BF16)}
    for k in grown:
        assert after[k] - before[k] == 32 << 20
    assert sizes() == before


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "_LIB_PATH", str(tmp_path / "libmonarch.so"))
    with pytest.raises(FileNotFoundError):
        B.lib()
