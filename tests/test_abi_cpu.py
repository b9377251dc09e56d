"""The C-ABI library loads without a GPU, exports every function include/rbs.h declares, and rejects bad
arguments on the host before anything would be launched (so these calls are safe on a CPU-only box)."""
import ctypes
import os
import re

import pytest

from paper_2609_20971_b200 import binding
from paper_2609_20971_b200.binding import RbsShape, RbsStats, RbsTensor

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
OK, INVALID, UNSUPPORTED, WORKSPACE = 0, 1, 2, 3


@pytest.fixture(scope="module")
def lib():
    from paper_2609_20971_b200.build import build_library
    build_library()
    return binding.load_library()


def declared_functions():
    names = []
    inc = os.path.join(ROOT, "include")
    for header in sorted(os.listdir(inc)):
        if header.endswith(".h"):
            names += re.findall(r"RBS_API\s+[\w\s\*]+?\b(rbs_\w+)\s*\(", open(os.path.join(inc, header)).read())
    return names


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"rbs_block_stats", "rbs_select", "rbs_sparse_prefill", "rbs_workspace_bytes",
            "rbs_selftest_device_table", "rbs_selftest_wait_timeout"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings_and_version(lib):
    assert lib.rbs_status_string(0) == b"RBS_OK"
    assert lib.rbs_status_string(2) == b"RBS_ERR_UNSUPPORTED"
    assert lib.rbs_status_string(6) == b"RBS_ERR_DEBUG_CHECK"
    assert b"sm_100a" in lib.rbs_version() and b"debug" not in lib.rbs_version()


def test_debug_library_builds_and_exports_the_same_symbols():
    """The variant with device-side index checks (-DRBS_DEBUG) is the same ABI: every declared symbol, and a version
    string that says which variant is loaded.  (Its checks run in the GPU tests.)"""
    import ctypes
    from paper_2609_20971_b200.build import build_library
    dbg = ctypes.CDLL(build_library(debug=True))
    for n in declared_functions():
        assert hasattr(dbg, n), n
    dbg.rbs_version.restype = ctypes.c_char_p
    assert b"debug checks" in dbg.rbs_version()
    # the self-test refuses a null flag before any launch (no GPU needed)
    dbg.rbs_selftest_debug_check.restype = ctypes.c_int
    dbg.rbs_selftest_debug_check.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
    assert dbg.rbs_selftest_debug_check(None, None) == INVALID


def _t(ptr=0x1000, sb=0, st=128, sh=128):
    return RbsTensor(ptr, sb, st, sh)


def _stats(v=0x1000):
    return RbsStats(v, v, v, v)


def test_shape_checks_reject_before_launch(lib):
    good = RbsShape(1, 1024, 4, 2, 128, 128)
    cases = [
        (RbsShape(1, 1024, 4, 2, 64, 128), UNSUPPORTED),    # head_dim
        (RbsShape(1, 1024, 4, 2, 128, 32), UNSUPPORTED),    # block size
        (RbsShape(1, 1024, 4, 2, 128, 512), UNSUPPORTED),
        (RbsShape(1, 1024, 3, 2, 128, 128), UNSUPPORTED),   # heads not divisible
        (RbsShape(0, 1024, 4, 2, 128, 128), INVALID),
    ]
    for shape, want in cases:
        assert lib.rbs_block_stats(ctypes.byref(shape), _t(), _stats(), None) == want
        assert lib.rbs_workspace_bytes(1, ctypes.byref(shape)) == 0
    assert lib.rbs_block_stats(None, _t(), _stats(), None) == INVALID
    assert lib.rbs_block_stats(ctypes.byref(good), _t(ptr=0), _stats(), None) == INVALID
    assert lib.rbs_block_stats(ctypes.byref(good), _t(ptr=0x1008), _stats(), None) == INVALID   # misaligned
    assert lib.rbs_block_stats(ctypes.byref(good), _t(st=100), _stats(), None) == INVALID       # stride % 8
    assert lib.rbs_block_stats(ctypes.byref(good), _t(), _stats(0), None) == INVALID


def test_select_argument_checks(lib):
    good = RbsShape(1, 1024, 4, 2, 128, 128)
    need = lib.rbs_workspace_bytes(1, ctypes.byref(good))
    assert need > 0 and need % 256 == 0
    p = ctypes.c_void_p(0x1000)

    def call(alpha_b=0.22, alpha_r=0.18, sink=1, mask=p, ws=p, ws_bytes=need):
        return lib.rbs_select(ctypes.byref(good), _t(), _stats(), alpha_b, alpha_r, sink, 1, 1, mask, p, None, None,
                              ws, ws_bytes, None)
    assert call(alpha_b=0.0) == INVALID
    assert call(alpha_r=-1.0) == INVALID
    assert call(sink=-1) == INVALID
    assert call(mask=None) == INVALID
    assert call(ws_bytes=need - 1) == WORKSPACE
    assert call(ws=ctypes.c_void_p(0x1010)) == WORKSPACE          # not 256-byte aligned


def test_prefill_argument_checks(lib):
    good = RbsShape(1, 1024, 4, 2, 128, 128)
    assert lib.rbs_sparse_prefill(ctypes.byref(good), _t(), _t(), _t(ptr=0), None, _t(), None, 0.0, None, 0, None) == INVALID
    assert lib.rbs_sparse_prefill(ctypes.byref(good), _t(), _t(), _t(), None, _t(), None, -1.0, None, 0, None) == INVALID


def test_prefill_workspace_checks(lib):
    good = RbsShape(1, 4096, 4, 2, 128, 128)
    need = lib.rbs_workspace_bytes(2, ctypes.byref(good))
    assert need > 0 and need % 256 == 0
    assert lib.rbs_workspace_bytes(2, ctypes.byref(RbsShape(1, 4096, 4, 2, 128, 64))) == 0   # blocks of 64: no schedule
    p = ctypes.c_void_p(0x1000)

    def call(mask=p, ws=p, ws_bytes=need):
        return lib.rbs_sparse_prefill(ctypes.byref(good), _t(), _t(), _t(), mask, _t(), None, 0.0, ws, ws_bytes, None)
    assert call(ws_bytes=need - 1) == WORKSPACE
    assert call(ws=ctypes.c_void_p(0x1010)) == WORKSPACE


def test_binding_fails_loudly_when_library_is_missing(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(binding.RbsError):
        binding.load_library()


def test_chunk_argument_checks(lib):
    good = RbsShape(1, 1000, 4, 2, 128, 128)          # M = 8, last block short
    need = lib.rbs_workspace_bytes(1, ctypes.byref(good))
    p = ctypes.c_void_p(0x1000)

    def sel(q0, nq):
        return lib.rbs_select_chunk(ctypes.byref(good), q0, nq, _t(), _stats(), 0.22, 0.18, 1, 1, 1, p, p, None, None,
                                    p, need, None)
    assert sel(-1, 128) == INVALID and sel(0, 0) == INVALID
    assert sel(7, 128) == INVALID                      # runs past the end of the sequence
    assert sel(2, 100) == INVALID                      # ends inside a block that is not the last
    assert lib.rbs_sparse_prefill_chunk(ctypes.byref(good), 8, 64, _t(), _t(), _t(), None, _t(), None, 0.0, None, 0,
                                        None) == INVALID


def test_group_union_argument_checks(lib):
    good = RbsShape(1, 1024, 4, 2, 128, 128)
    p = ctypes.c_void_p(0x1000)
    lib.rbs_mask_group_union.argtypes = [ctypes.POINTER(RbsShape), ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
                                         ctypes.c_void_p, ctypes.c_void_p]
    assert lib.rbs_mask_group_union(ctypes.byref(good), 0, -1, None, p, None) == INVALID
    assert lib.rbs_mask_group_union(ctypes.byref(good), 0, -1, p, None, None) == INVALID
    assert lib.rbs_mask_group_union(ctypes.byref(good), 7, 256, p, p, None) == INVALID      # past the end
    bad = RbsShape(1, 1024, 3, 2, 128, 128)
    assert lib.rbs_mask_group_union(ctypes.byref(bad), 0, -1, p, p, None) == UNSUPPORTED


def test_per_device_lookup_table(lib):
    """Values such as the device address of the status word are looked up once per device and never handed to
    another device: the table logic is host-only and is checked here with a fake lookup (0 = every check passed)."""
    assert lib.rbs_selftest_device_table() == 0


def test_wait_timeout_selftest_argument_checks(lib):
    p = ctypes.c_void_p(0x1000)
    assert lib.rbs_selftest_wait_timeout(0, p, None) == INVALID
    assert lib.rbs_selftest_wait_timeout(1 << 20, p, None) == INVALID      # only short limits are accepted
    assert lib.rbs_selftest_wait_timeout(1024, None, None) == INVALID


def test_varlen_argument_checks(lib):
    lib.rbs_varlen_workspace_bytes.restype = ctypes.c_size_t
    good = (ctypes.c_int * 4)(0, 300, 1000, 1001)
    need = lib.rbs_varlen_workspace_bytes(3, good, 4, 2, 128, 128)
    assert need > 0 and need % 256 == 0
    assert lib.rbs_varlen_workspace_bytes(3, (ctypes.c_int * 4)(1, 300, 1000, 1001), 4, 2, 128, 128) == 0     # not from 0
    assert lib.rbs_varlen_workspace_bytes(3, (ctypes.c_int * 4)(0, 300, 300, 1001), 4, 2, 128, 128) == 0      # empty prompt
    assert lib.rbs_varlen_workspace_bytes(3, good, 4, 2, 64, 128) == 0                                          # head_dim
    p = ctypes.c_void_p(0x1000)
    t = _t()
    assert lib.rbs_prefill_varlen(3, good, 4, 2, 128, 128, t, t, t, t, 0.22, 0.18, 1, 1, 1, p, p, need - 1, None) == WORKSPACE
    assert lib.rbs_prefill_varlen(3, good, 4, 2, 128, 128, t, t, t, t, 0.22, 0.18, 1, 1, 1, None, p, need, None) == INVALID
    assert lib.rbs_prefill_varlen(0, good, 4, 2, 128, 128, t, t, t, t, 0.22, 0.18, 1, 1, 1, p, p, need, None) == INVALID


def test_grouped_prefill_and_box_selector_argument_checks(lib):
    p = ctypes.c_void_p(0x1000)
    t = _t()
    lib.rbs_sparse_prefill_grouped.restype = ctypes.c_int
    good = RbsShape(1, 1024, 4, 2, 128, 128)
    assert lib.rbs_sparse_prefill_grouped(ctypes.byref(good), t, t, t, None, t, None, ctypes.c_float(0.0), None) == INVALID   # needs a mask
    odd = RbsShape(1, 1024, 3, 1, 128, 128)                       # group of three heads: no pairs
    assert lib.rbs_sparse_prefill_grouped(ctypes.byref(odd), t, t, t, p, t, None, ctypes.c_float(0.0), None) == UNSUPPORTED
    b64 = RbsShape(1, 1024, 4, 2, 128, 64)
    assert lib.rbs_sparse_prefill_grouped(ctypes.byref(b64), t, t, t, p, t, None, ctypes.c_float(0.0), None) == UNSUPPORTED
    box = binding.RbsBox(0x1000, 0x1000)
    need = lib.rbs_workspace_bytes(3, ctypes.byref(good))
    assert need > 0 and lib.rbs_workspace_bytes(3, ctypes.byref(RbsShape(1, 1024, 4, 2, 128, 256))) == 0
    call = lambda shape, delta, ws_bytes=need: lib.rbs_select_box(ctypes.byref(shape), t, box, ctypes.c_double(delta), 1, 1, 1, p, p,
                                                                  None, p, ws_bytes, None)
    assert call(good, 0.0) == INVALID and call(good, 1.5) == INVALID
    assert call(good, 0.05, need - 1) == WORKSPACE
    assert call(RbsShape(1, 1024, 4, 2, 128, 256), 0.05) == UNSUPPORTED
    assert lib.rbs_block_stats_box(ctypes.byref(good), t, _stats(), binding.RbsBox(0, 0x1000), None) == INVALID
