"""The C-ABI library builds for sm_100a, loads, and exports every symbol that include/*.h
declares.  Only host-side calls are made here (size queries, status strings, argument checks
that return before any CUDA call)."""
import ctypes
import glob
import os
import re

import pytest

from paper_2601_15498_b200 import build, mars

import hookctl as hooks

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = []
    for h in sorted(glob.glob(os.path.join(ROOT, "include", "*.h"))):
        src = open(h).read()
        src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
        names += re.findall(r"\b(mars_[a-z0-9_]+)\s*\(", src)
    return sorted(set(names))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return mars.lib()


def test_library_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert {"mars_verify_chain", "mars_verify_tree", "mars_workspace_bytes",
            "mars_status_string"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
        getattr(lib, n)


def test_status_strings(lib):
    seen = {lib.mars_status_string(c) for c in range(5)}
    assert len(seen) == 5 and all(s for s in seen)
    assert lib.mars_status_string(99) == b"unknown status"


def test_workspace_bytes_host_only(lib, monkeypatch):
    hooks.clear("HOOK_FORCE_SPLIT")
    wb = lib.mars_workspace_bytes
    assert wb(0, 1, 100, 0) == 0 and wb(1, 0, 100, 0) == 0 and wb(1, 1, 1, 0) == 0
    assert wb(1, 1025, 100, 0) == 0 and wb(1, 1, 100, 7) == 0
    # whole rows per block once the batch fills the GPU: one 16-byte record per row + counters
    assert wb(256, 60, 151936, 0) == 1024 + 256 * 60 * 16
    # few rows: rows are split, the workspace grows with the number of slices
    small = wb(1, 6, 32000, 1)
    assert small % 16 == 0 and 256 + 6 * 16 < small <= 256 + 6 * 16 * 64
    assert wb(1, 60, 151936, 0) > 256 + 60 * 16
    hooks.set("HOOK_FORCE_SPLIT", 3)
    assert wb(2, 5, 4000, 1) == 256 + 10 * 3 * 16


def test_argument_checks_return_before_any_cuda_call(lib):
    """NULL pointers and bad sizes are rejected on the host (no GPU is needed to see that)."""
    n = None
    dummy = ctypes.c_void_p(256)
    assert lib.mars_verify_tree(n, 10, 0, n, n, 1, 1, 10, 0.9, 0, n, n, n, n, 0, n, None, n, 0, n) == 1
    assert lib.mars_verify_chain(dummy, 10, 0, dummy, 0, 2, 10, 0.9, 0, dummy, dummy, dummy, n, None,
                                 dummy, 1 << 20, n) == 1
    # ld < V
    assert lib.mars_verify_chain(dummy, 5, 0, dummy, 1, 2, 10, 0.9, 0, dummy, dummy, dummy, n, None,
                                 dummy, 1 << 20, n) == 1
    # NaN theta
    assert lib.mars_verify_chain(dummy, 10, 0, dummy, 1, 2, 10, float("nan"), 0, dummy, dummy, dummy,
                                 n, None, dummy, 1 << 20, n) == 1
    # unknown flag / too many nodes / unknown dtype
    assert lib.mars_verify_chain(dummy, 10, 0, dummy, 1, 2, 10, 0.9, 1024, dummy, dummy, dummy, n, None,
                                 dummy, 1 << 20, n) == 3
    assert lib.mars_verify_chain(dummy, 10, 0, dummy, 1, 2000, 10, 0.9, 0, dummy, dummy, dummy, n, None,
                                 dummy, 1 << 20, n) == 3
    assert lib.mars_verify_chain(dummy, 10, 5, dummy, 1, 2, 10, 0.9, 0, dummy, dummy, dummy, n, None,
                                 dummy, 1 << 20, n) == 3
    # workspace: missing, too small, misaligned
    assert lib.mars_verify_chain(dummy, 10, 0, dummy, 1, 2, 10, 0.9, 0, dummy, dummy, dummy, n, None,
                                 n, 0, n) == 2
    assert lib.mars_verify_chain(dummy, 10, 0, dummy, 1, 2, 10, 0.9, 0, dummy, dummy, dummy, n, None,
                                 dummy, 16, n) == 2
    assert lib.mars_verify_chain(dummy, 10, 0, dummy, 1, 2, 10, 0.9, 0, dummy, dummy, dummy, n, None,
                                 ctypes.c_void_p(260), 1 << 20, n) == 2
    # misaligned logits pointer for the element size
    assert lib.mars_verify_chain(ctypes.c_void_p(257), 10, 1, dummy, 1, 2, 10, 0.9, 0, dummy, dummy,
                                 dummy, n, None, dummy, 1 << 20, n) == 1


def test_missing_library_is_an_error(monkeypatch, tmp_path):
    monkeypatch.setattr(mars, "_lib", None)
    monkeypatch.setattr(build, "LIB", str(tmp_path / "nope.so"))
    with pytest.raises(mars.MarsError, match="no fallback"):
        mars.lib()


def test_hooks_are_set_only_through_the_abi(lib, monkeypatch):
    """The library ignores the environment; a hook is a process-wide integer behind
    mars_test_hook, which returns the previous value and rejects unknown hooks."""
    wb = lib.mars_workspace_bytes
    plain = wb(2, 5, 4000, 1)
    monkeypatch.setenv("MARS_FORCE_SPLIT", "3")
    assert wb(2, 5, 4000, 1) == plain
    assert lib.mars_test_hook(0, 3) == 0
    assert wb(2, 5, 4000, 1) == 256 + 10 * 3 * 16
    assert lib.mars_test_hook(0, 0) == 3
    assert wb(2, 5, 4000, 1) == plain
    assert lib.mars_test_hook(5, 1) == -1 and lib.mars_test_hook(-1, 1) == -1 and lib.mars_test_hook(0, -2) == -1


@pytest.mark.skipif(__import__("torch").cuda.is_available(), reason="host without a GPU only")
def test_device_check_reports_a_missing_device(lib):
    sm, tuned = ctypes.c_int(-1), ctypes.c_int(-1)
    assert lib.mars_device_check(ctypes.byref(sm), ctypes.byref(tuned)) == 4      # MARS_ERR_CUDA
    assert tuned.value == 148


def test_binding_declares_every_exported_function(lib):
    """The Python binding states argument and result types for every function of the header, so
    that no call goes through ctypes' int-sized defaults (which would truncate 64-bit pointers)."""
    for n in declared_functions():
        fn = getattr(lib, n)
        assert fn.argtypes is not None, n


def test_host_buffer_entry_point_checks_its_arguments_on_the_host(lib):
    n = None
    p = ctypes.c_void_p(4096)
    size = lib.mars_verify_tree_host_staging_bytes
    assert size(0, 3, 100, 0, 100, 2) == 0 and size(2, 3, 100, 0, 50, 2) == 0 and size(2, 3, 100, 7, 100, 2) == 0
    need = size(2, 3, 100, 1, 104, 2)
    # logits 2*3*104*4 B, tokens and parents, five result arrays, workspace: each rounded up to 256 B
    assert need % 256 == 0 and need >= 2 * 3 * 104 * 4 + lib.mars_workspace_bytes(2, 3, 100, 1)
    call = lib.mars_verify_tree_host
    assert call(n, 104, 1, p, p, 2, 3, 100, 0.9, 0, p, p, n, p, 2, n, p, need, n) == 1          # NULL logits
    assert call(p, 104, 1, p, p, 2, 3, 100, float("nan"), 0, p, p, n, p, 2, n, p, need, n) == 1  # NaN theta
    assert call(p, 104, 1, p, p, 2, 3, 100, 0.9, 4, p, p, n, p, 2, n, p, need, n) == 3            # flag not taken here
    assert call(p, 104, 1, p, p, 2, 3, 100, 0.9, 0, p, p, n, p, 2, n, p, need - 1, n) == 2        # staging too small
    assert call(p, 104, 1, p, p, 2, 3, 100, 0.9, 0, p, p, n, p, 2, n, ctypes.c_void_p(4100), need, n) == 2
