"""The C-ABI library loads without a GPU and exports every symbol the header
declares; argument errors are reported before any device work."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    import importlib.util

    spec = importlib.util.spec_from_file_location("_mmv_build", ROOT / "paper_2506_23906_b200" / "build.py")
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return ctypes.CDLL(str(mod.build()))


def declared_symbols():
    text = (ROOT / "include" / "mmv.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mmv_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_entry_points():
    syms = declared_symbols()
    for s in ("mmv_seg_scan", "mmv_seg_sum", "mmv_spmv_csr", "mmv_workspace_bytes",
              "mmv_last_async_status", "mmv_status_string"):
        assert s in syms


def test_every_declared_symbol_is_exported(lib):
    for s in declared_symbols():
        assert hasattr(lib, s), f"{s} declared in include/mmv.h but not exported"


def test_binding_lists_the_same_symbols():
    src = (ROOT / "paper_2506_23906_b200" / "__init__.py").read_text()
    for s in declared_symbols():
        assert f'"{s}"' in src or f"lib.{s}" in src


def test_host_only_calls(lib):
    lib.mmv_status_string.restype = ctypes.c_char_p
    assert lib.mmv_status_string(0) == b"ok"
    assert b"timed out" in lib.mmv_status_string(5)
    lib.mmv_workspace_bytes.restype = ctypes.c_size_t
    lib.mmv_workspace_bytes.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int64, ctypes.c_int64]
    assert lib.mmv_workspace_bytes(0, 0, 0, -1, 0) == 0
    assert lib.mmv_workspace_bytes(7, 0, 0, 10, 0) == 0
    small = lib.mmv_workspace_bytes(0, 0, 0, 1, 0)
    big = lib.mmv_workspace_bytes(0, 0, 0, 1 << 30, 0)
    assert 256 < small <= 1024 and (1 << 21) <= big <= (1 << 22)       # 8 bytes per 4096 elements (a tile of 16384 uses every fourth word)
    # an offset-encoded scan also needs n scratch flag bytes; SpMV needs 4 bytes per non-zero
    assert lib.mmv_workspace_bytes(0, 0, 1, 1 << 20, 10) >= small + (1 << 20)
    assert lib.mmv_workspace_bytes(2, 0, 1, 1 << 20, 10) >= 4 << 20


def test_argument_errors_are_synchronous(lib):
    vp, i64, sz, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t, ctypes.c_int
    lib.mmv_seg_scan.argtypes = [vp, vp, ci, i64, i64, ci, vp, vp, sz, vp]
    lib.mmv_seg_sum.argtypes = [vp, vp, ci, i64, i64, ci, vp, vp, vp, sz, vp]
    lib.mmv_spmv_csr.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, vp, sz, vp]
    assert lib.mmv_seg_scan(None, None, 0, -1, 0, 0, None, None, 0, None) == 1      # negative n
    assert lib.mmv_seg_scan(None, None, 0, 0, 0, 0, None, None, 0, None) == 0       # n == 0: nothing to do
    assert lib.mmv_seg_scan(None, None, 0, 8, 0, 0, None, None, 0, None) == 1       # null pointers
    assert lib.mmv_seg_scan(16, 16, 0, 8, 0, 9, 16, 256, 4096, None) == 1           # bad dtype
    assert lib.mmv_seg_scan(16, 16, 3, 8, 0, 0, 16, 256, 4096, None) == 1           # bad segment format
    assert lib.mmv_seg_scan(18, 16, 0, 8, 0, 0, 16, 256, 4096, None) == 1           # misaligned x
    assert lib.mmv_seg_scan(16, 16, 0, 8, 0, 0, 16, 256, 16, None) == 3             # workspace too small
    lib.mmv_seg_scan_exclusive.argtypes = lib.mmv_seg_scan.argtypes
    assert lib.mmv_seg_scan_exclusive(None, None, 0, -1, 0, 0, None, None, 0, None) == 1      # negative n
    assert lib.mmv_seg_scan_exclusive(None, None, 0, 0, 0, 2, None, None, 0, None) == 0       # n == 0, bf16: nothing to do
    assert lib.mmv_seg_scan_exclusive(16, 16, 0, 8, 0, 3, 16, 256, 4096, None) == 1           # bad dtype
    assert lib.mmv_seg_scan(16, 16, 0, 8, 0, 2, 16, 256, 16, None) == 3                       # bf16 accepted: workspace too small
    assert lib.mmv_seg_sum(None, None, 1, 0, 0, 0, None, None, None, 0, None) == 0  # nothing to do
    assert lib.mmv_seg_sum(16, 16, 1, -5, 1, 0, 16, None, 256, 4096, None) == 1
    assert lib.mmv_seg_sum(16, 16, 1, 8, (1 << 31) - 1, 0, 16, None, 256, 1 << 40, None) == 1   # more segments than 32-bit indices hold
    assert lib.mmv_spmv_csr(16, 16, 16, 16, 16, (1 << 31) - 1, 8, 8, 256, 1 << 40, None) == 1    # ... or rows
    assert lib.mmv_seg_sum(16, 16, 0, 8, 0, 0, 16, None, 256, 16, None) == 3        # flag form: workspace too small
    assert lib.mmv_seg_sum(16, 16, 0, 8, 0, 0, 16, 12, 256, 1 << 20, None) == 1     # misaligned segment counter
    lib.mmv_seg_scan_host.argtypes = [vp, vp, i64, ci, vp, i64, vp, sz, vp]
    lib.mmv_seg_scan_host_scratch_bytes.restype = sz
    lib.mmv_seg_scan_host_scratch_bytes.argtypes = [ci, i64]
    assert lib.mmv_seg_scan_host(16, 16, 8, 0, 16, 1000, 256, 1 << 30, None) == 1     # chunk not a multiple of 16384
    assert lib.mmv_seg_scan_host(16, 16, 8, 0, 16, 16384, 256, 16, None) == 3         # scratch too small
    assert lib.mmv_seg_scan_host(None, None, 0, 0, None, 16384, None, 0, None) == 0   # nothing to do
    assert lib.mmv_seg_scan_host(16, 16, 8, 2, 16, 16384, 256, 1 << 30, None) == 1    # bf16 values: not for this entry point
    assert lib.mmv_seg_scan_host_scratch_bytes(0, 1000) == 0
    assert lib.mmv_seg_scan_host_scratch_bytes(0, 16384) >= 2 * 16384 * 7
    lib.mmv_compress.argtypes = [vp, vp, i64, ci, vp, vp, vp, sz, vp]
    assert lib.mmv_compress(None, None, 0, 0, None, None, None, 0, None) == 0           # nothing to do
    assert lib.mmv_compress(None, None, -1, 0, None, None, None, 0, None) == 1
    assert lib.mmv_compress(16, 16, 8, 0, 16, None, 256, 16, None) == 3                 # workspace too small
    assert lib.mmv_compress(16, 16, 8, 0, 16, 12, 256, 1 << 20, None) == 1              # misaligned counter
    assert lib.mmv_workspace_bytes(3, 0, 0, 1 << 20, 0) >= 512
    lib.mmv_seg_scan_minmax.argtypes = [vp, vp, i64, ci, ci, vp, vp, sz, vp]
    assert lib.mmv_seg_scan_minmax(None, None, 0, 0, 0, None, None, 0, None) == 0          # nothing to do
    assert lib.mmv_seg_scan_minmax(None, None, -1, 0, 0, None, None, 0, None) == 1
    assert lib.mmv_seg_scan_minmax(16, 16, 8, 3, 0, 16, 256, 1 << 20, None) == 1           # bad dtype
    assert lib.mmv_seg_scan_minmax(16, 16, 8, 2, 0, 16, 256, 16, None) == 3                # bf16 accepted: workspace too small
    assert lib.mmv_seg_scan_minmax(16, 16, 8, 0, 1, 16, 256, 16, None) == 3                # workspace too small
    assert lib.mmv_seg_scan_minmax(16, 18, 8, 0, 1, 16, 256, 1 << 20, None) == 1           # misaligned flags
    assert lib.mmv_workspace_bytes(4, 0, 0, 1 << 20, 0) >= 256 * 8
    lib.mmv_seg_scan_i8_i64.argtypes = [vp, vp, i64, vp, vp, sz, vp]
    assert lib.mmv_seg_scan_i8_i64(None, None, 0, None, None, 0, None) == 0                # nothing to do
    assert lib.mmv_seg_scan_i8_i64(None, None, -1, None, None, 0, None) == 1
    assert lib.mmv_seg_scan_i8_i64(16, 16, 8, 16, 256, 16, None) == 3                      # workspace too small
    assert lib.mmv_seg_scan_i8_i64(16, 16, 8, 24, 256, 1 << 20, None) == 1                 # misaligned output
    assert lib.mmv_workspace_bytes(5, 1, 0, 1 << 20, 0) >= 256 * 32
    assert lib.mmv_spmv_csr(None, None, None, None, None, -1, 1, 1, None, 0, None) == 1
    assert lib.mmv_spmv_csr(None, None, None, None, None, 0, 1, 0, None, 0, None) == 0
