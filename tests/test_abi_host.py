"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the header
declares, and rejects bad arguments before launching anything."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2208_11580_b200 import build, binding
    build.build()
    return binding.load_library()


def test_exports_every_declared_symbol(lib):
    from paper_2208_11580_b200 import binding
    header = open(os.path.join(ROOT, "include", "obc.h")).read()
    declared = set(re.findall(r"\b(obc_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTED_SYMBOLS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_status_strings(lib):
    from paper_2208_11580_b200 import obc_status_string
    seen = {obc_status_string(i) for i in range(10)}
    assert len(seen) == 10 and "ok" in seen
    assert obc_status_string(12345) == "unknown status"


def test_argument_errors_return_before_any_launch(lib):
    f = ctypes.c_void_p
    good = f(0x1000)
    # NULL / negative / inconsistent sizes
    assert lib.obc_hessian(None, 8, 16, 16, good, 8, 0, 0, None, 0, good, 1 << 30, None) == 1
    assert lib.obc_hessian(good, 8, 16, 8, good, 8, 0, 0, None, 0, good, 1 << 30, None) == 1       # ldx < n
    assert lib.obc_hessian(good, 8, 16, 16, good, 8, 2, 0, None, 0, good, 1 << 30, None) == 1       # accumulate flag
    assert lib.obc_hessian(good, 8, 16, 16, good, 8, 0, 9, None, 0, good, 1 << 30, None) == 1       # precision enum
    assert lib.obc_hessian(f(0x1004), 8, 16, 16, good, 8, 0, 0, None, 0, good, 1 << 30, None) == 2  # misaligned X
    assert lib.obc_hessian(good, 8, 16, 18, good, 8, 0, 0, None, 0, good, 1 << 30, None) == 2       # ldx % 4
    assert lib.obc_hessian(good, 8, 16, 16, good, 8, 0, 0, None, 0, None, 0, None) == 3    # no workspace
    assert lib.obc_hessian(good, 8, 16, 16, good, 8, 0, 0, None, 0, good, 16, None) == 3   # too small
    assert lib.obc_hessian_inverse(good, 8, 8, ctypes.c_float(-1.0), good, 8, good, good, 1 << 30, None) == 1
    assert lib.obc_hessian_inverse(good, 8, 8, ctypes.c_float(0.01), good, 8, None, good, 1 << 30, None) == 1
    assert lib.obc_hessian_inverse(good, 8, 8, ctypes.c_float(0.01), good, 8, good, good, 64, None) == 3
    assert lib.obc_prune_trace(good, 8, 4, 8, 2, 3, good, 8, 8, good, good, None, good, good, 1 << 30, None, None) == 1  # rows
    assert lib.obc_prune_trace(good, 8, 4, 8, 0, 4, good, 8, 9, good, good, None, good, good, 1 << 30, None, None) == 1  # steps
    assert lib.obc_prune_trace(good, 8, 4, 8, 0, 4, good, 8, 8, None, good, None, good, good, 1 << 30, None, None) == 1
    assert lib.obc_prune_trace(good, 6000, 4, 6000, 0, 4, good, 6000, 8, good, good, None, good, good, 1 << 30, None, None) == 8
    assert lib.obc_prune_trace(good, 10, 4, 8, 0, 4, good, 8, 8, good, good, None, good, good, 1 << 30, None, None) == 2
    assert lib.obc_select_global_mask(good, good, 4, 8, 33, good, good, good, 1 << 30, None) == 1   # k > d_row*d_col
    assert lib.obc_select_global_mask(good, good, 4, 8, -1, good, good, good, 1 << 30, None) == 1
    assert lib.obc_select_global_mask(good, good, 4, 8, 5, good, good, good, 8, None) == 3
    st = lib.obc_select_global_mask_static
    assert st(good, good, 4, 8, 33, good, good, None) == 1                                           # k out of range
    assert st(good, good, 20000, 8, 5, good, good, None) == 9                                        # rows over the built-in limit
    assert st(good, good, 4096, 2048, 5, good, good, None) == 9                                      # entries over the limit
    assert lib.obc_minmax_grid(good, 8, 4, 8, None, 1, 0, good, good, None, None) == 1              # bits
    assert lib.obc_minmax_grid(good, 8, 4, 8, None, 4, 2, good, good, None, None) == 1              # symmetric flag
    q = lib.obc_quantize
    assert q(good, 8, 4, 8, 0, 4, good, 8, good, good, 4, 0, good, None, 0, good, 8, good, None, None, good, good, 1 << 30, None, None) == 1
    assert q(good, 8, 4, 8, 0, 4, good, 8, good, good, 4, 0, None, None, 4, good, 8, good, None, None, good, good, 1 << 30, None, None) == 1
    assert q(good, 8, 4, 8, 0, 4, good, 8, None, good, 4, 0, None, None, 0, good, 8, good, None, None, good, good, 1 << 30, None, None) == 1
    assert lib.obc_prune_apply(good, 8, 4, 8, 0, 4, good, 8, good, None, None, 0, good, 8, good, good, 1 << 30, None, None) == 1
    assert lib.obc_prune_apply(good, 8, 4, 8, 0, 4, good, 8, good, good, good, 0, good, 8, good, good, 1 << 30, None, None) == 1


def test_engine_options_are_validated_per_call(lib):
    """the per-call engine options are checked on the host like every other argument (no process-wide engine state)"""
    from paper_2208_11580_b200 import binding
    good = ctypes.c_void_p(0x1000)
    def trace(opts):
        return lib.obc_prune_trace(good, 8, 4, 8, 0, 4, good, 8, 8, good, good, None, good, None, 0,
                                   binding._opts(opts), None)
    assert trace(binding.EngineOpts(7, 0, 0, 0)) == 1          # unknown engine
    assert trace(binding.EngineOpts(2, 100, 0, 0)) == 1        # threads not 128/256/512
    assert trace(binding.EngineOpts(2, 0, 65, 0)) == 1         # more deferred updates than the kernels hold
    assert trace(binding.EngineOpts(2, 0, 0, 2)) == 1          # unknown flag
    plan = (ctypes.c_int32 * 8)()
    assert lib.obc_engine_plan(8, 0, 0, binding._opts(binding.EngineOpts(9, 0, 0, 0)), plan) == 1
    assert "obc_set_engine" not in binding.EXPORTED_SYMBOLS


def test_workspace_queries_on_host(lib):
    from paper_2208_11580_b200 import obc_workspace_bytes, OP_HESSIAN, OP_INVERSE, OP_SELECT
    assert obc_workspace_bytes(OP_INVERSE, 0, 3072) >= 3 * 3072 * 3072 * 8
    assert obc_workspace_bytes(OP_SELECT, 768, 3072) >= 768 * 3072 * 4
    assert obc_workspace_bytes(OP_HESSIAN, 0, 576, 16384) >= 576 * 576 * 4
    assert obc_workspace_bytes(OP_HESSIAN, 0, 0, 16384) == 0
    assert obc_workspace_bytes(99, 1, 8) == 0


def test_missing_library_fails_loudly(monkeypatch):
    from paper_2208_11580_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIBPATH", "/nonexistent/libobc.so")
    with pytest.raises(RuntimeError, match="missing"):
        binding.load_library()
