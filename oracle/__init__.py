"""Python face of the CPU oracle (``oracle/mmv_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the test-suite, by the smoke check and by
the benchmark's CPU-baseline / reference legs, never by the GPU library.  The
module compiles the C file with gcc on first use (``build()``) and exposes thin
numpy wrappers; all arithmetic lives in the C file, which states the paper's
definitions (Problem 2.1 / Eq. 1, the segmented-sum definition of Section 2,
Algorithm 4.4 for CSR SpMV).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "mmv_oracle.c"
_SRC_PAR = _HERE / "mmv_oracle_par.c"
_LIB = _HERE / "libmmv_oracle.so"
_lib = None

# Tolerance of the fp16 -> fp32 paths: |gpu - oracle| <= REL * a + ABS where a is
# the sum of |x| over the same range the result sums over.
TOL_REL = 2e-3
TOL_ABS = 1e-6


def build(force: bool = False) -> Path:
    """Compile the oracle's C file into a shared library next to it."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < max(_SRC.stat().st_mtime, _SRC_PAR.stat().st_mtime):
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.run(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fno-fast-math", "-pthread",
             "-o", str(tmp), str(_SRC), str(_SRC_PAR), "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(str(_LIB))
        _lib.mmv_oracle_half_to_double.restype = ctypes.c_double
        _lib.mmv_oracle_half_to_double.argtypes = [ctypes.c_uint16]
        _lib.mmv_oracle_seg_sum_flags_f16.restype = ctypes.c_int64
        _lib.mmv_oracle_seg_sum_flags_i8.restype = ctypes.c_int64
        _lib.mmv_oracle_flags_from_offsets.restype = ctypes.c_int
    return _lib


def _p(a):
    return None if a is None else ctypes.c_void_p(a.ctypes.data)


def _as_f16_bits(x) -> np.ndarray:
    x = np.ascontiguousarray(x)
    if x.dtype == np.float16:
        return x.view(np.uint16)
    if x.dtype == np.uint16:
        return x
    raise TypeError("fp16 values must be float16 (or their uint16 bit patterns)")


def _as(x, dt) -> np.ndarray:
    x = np.ascontiguousarray(x)
    if x.dtype != dt:
        raise TypeError(f"expected {dt}, got {x.dtype}")
    return x


def half_to_double(bits: int) -> float:
    return float(_load().mmv_oracle_half_to_double(int(bits)))


def seg_scan_f16(x, f, state=None):
    """Eq. (1) on fp16 values: returns (z, a) in float64.

    ``state`` (a 2-element float64 array) continues an earlier chunk and is
    updated in place, so long inputs can be streamed.
    """
    xb, fb = _as_f16_bits(x), _as(f, np.uint8)
    n = xb.shape[0]
    assert fb.shape[0] == n
    z = np.empty(n, np.float64)
    a = np.empty(n, np.float64)
    has_prev = 0
    st = None
    if state is not None:
        st = _as(state["v"], np.float64)
        has_prev = int(state["open"])
    else:
        st = np.zeros(2, np.float64)
    _load().mmv_oracle_seg_scan_f16(_p(xb), _p(fb), ctypes.c_int64(n), _p(z), _p(a),
                                    ctypes.c_int(has_prev), _p(st))
    if state is not None and n > 0:
        state["open"] = True
    return z, a


def seg_scan_f16_all_cores(x, f, threads: int | None = None):
    """Eq. (1) on fp16 values, chunk-parallel over `threads` host threads (default: the cores this
    process may use) with a sequential carry hand-over between the chunks.  Returns (z, a, threads used)."""
    xb, fb = _as_f16_bits(x), _as(f, np.uint8)
    n = xb.shape[0]
    assert fb.shape[0] == n
    if threads is None:
        threads = len(os.sched_getaffinity(0))
    z = np.empty(n, np.float64)
    a = np.empty(n, np.float64)
    used = _load().mmv_oracle_seg_scan_f16_chunks(_p(xb), _p(fb), ctypes.c_int64(n), _p(z), _p(a), ctypes.c_int(int(threads)))
    if used <= 0:
        raise MemoryError("mmv_oracle_seg_scan_f16_chunks")
    return z, a, int(used)


def new_f16_state():
    return {"v": np.zeros(2, np.float64), "open": False}


def seg_scan_i8(x, f, state=None):
    """Eq. (1) on int8 values, int32 result (low 32 bits of the exact sum)."""
    xb, fb = _as(x, np.int8), _as(f, np.uint8)
    n = xb.shape[0]
    assert fb.shape[0] == n
    z = np.empty(n, np.int32)
    has_prev = 0
    if state is not None:
        st = _as(state["v"], np.int64)
        has_prev = int(state["open"])
    else:
        st = np.zeros(1, np.int64)
    _load().mmv_oracle_seg_scan_i8(_p(xb), _p(fb), ctypes.c_int64(n), _p(z),
                                   ctypes.c_int(has_prev), _p(st))
    if state is not None and n > 0:
        state["open"] = True
    return z


def new_i8_state():
    return {"v": np.zeros(1, np.int64), "open": False}


def seg_scan_excl_f16(x, f):
    """Segmented exclusive scan on fp16 values: e(i) = sum of the elements of i's segment in front
    of i (0 at a segment start); returns (e, a) in float64, a = the same sum over |x|."""
    xb, fb = _as_f16_bits(x), _as(f, np.uint8)
    n = xb.shape[0]
    assert fb.shape[0] == n
    e = np.empty(n, np.float64)
    a = np.empty(n, np.float64)
    _load().mmv_oracle_seg_scan_excl_f16(_p(xb), _p(fb), ctypes.c_int64(n), _p(e), _p(a))
    return e, a


def seg_scan_i8_wide(x, f) -> np.ndarray:
    """Eq. (1) on int8 values with an int64 result: the exact sums, no wrap."""
    xb, fb = _as(x, np.int8), _as(f, np.uint8)
    n = xb.shape[0]
    assert fb.shape[0] == n
    z = np.empty(n, np.int64)
    _load().mmv_oracle_seg_scan_i8_wide(_p(xb), _p(fb), ctypes.c_int64(n), _p(z))
    return z


def seg_scan_minmax_f16(x, f, want_min: bool = False) -> np.ndarray:
    """Segmented running maximum (or minimum) of fp16 values, float64 (exact: no arithmetic is involved)."""
    xb, fb = _as_f16_bits(x), _as(f, np.uint8)
    n = xb.shape[0]
    assert fb.shape[0] == n
    z = np.empty(n, np.float64)
    _load().mmv_oracle_seg_scan_minmax_f16(_p(xb), _p(fb), ctypes.c_int64(n), ctypes.c_int(int(want_min)), _p(z))
    return z


def seg_scan_minmax_bf16(xbits, f, want_min: bool = False) -> np.ndarray:
    """Segmented running maximum (or minimum) of bfloat16 values given as uint16 bit patterns, float64 (exact)."""
    x, fb = bf16_to_double(xbits), _as(f, np.uint8)
    n = x.shape[0]
    assert fb.shape[0] == n
    z = np.empty(n, np.float64)
    _load().mmv_oracle_seg_scan_minmax_f64(_p(x), _p(fb), ctypes.c_int64(n), ctypes.c_int(int(want_min)), _p(z))
    return z


def seg_scan_minmax_i8(x, f, want_min: bool = False) -> np.ndarray:
    xb, fb = _as(x, np.int8), _as(f, np.uint8)
    n = xb.shape[0]
    assert fb.shape[0] == n
    z = np.empty(n, np.int32)
    _load().mmv_oracle_seg_scan_minmax_i8(_p(xb), _p(fb), ctypes.c_int64(n), ctypes.c_int(int(want_min)), _p(z))
    return z


def compress(x, f) -> np.ndarray:
    """COMPRESS (Section 2): the elements x(i) with f(i) != 0, in order, copied unchanged."""
    x = np.ascontiguousarray(x)
    fb = _as(f, np.uint8)
    assert fb.shape[0] == x.shape[0]
    out = np.empty_like(x)
    lib = _load()
    lib.mmv_oracle_compress.restype = ctypes.c_int64
    k = lib.mmv_oracle_compress(_p(x.view(np.uint8)), _p(fb), ctypes.c_int64(x.shape[0]), ctypes.c_int(x.dtype.itemsize),
                                _p(out.view(np.uint8)))
    return out[:k].copy()


def bf16_to_double(bits) -> np.ndarray:
    """Exact decode of bfloat16 bit patterns (uint16) to float64."""
    hb = _as(bits, np.uint16)
    out = np.empty(hb.shape[0], np.float64)
    _load().mmv_oracle_decode_bf16(_p(hb), ctypes.c_int64(hb.shape[0]), _p(out))
    return out


def seg_scan_bf16(xbits, f, exclusive: bool = False):
    """Eq. (1) (or its exclusive companion) on bfloat16 values given as uint16 bit patterns: (z, a) in float64."""
    x, fb = bf16_to_double(xbits), _as(f, np.uint8)
    n = x.shape[0]
    assert fb.shape[0] == n
    z, a = np.empty(n, np.float64), np.empty(n, np.float64)
    fn = _load().mmv_oracle_seg_scan_excl_f64 if exclusive else _load().mmv_oracle_seg_scan_f64
    fn(_p(x), _p(fb), ctypes.c_int64(n), _p(z), _p(a))
    return z, a


def seg_sum_csr_bf16(xbits, off):
    x, off = bf16_to_double(xbits), _as(off, np.int32)
    _check_offsets(off, x.shape[0])
    nseg = off.shape[0] - 1
    out, a = np.empty(nseg, np.float64), np.empty(nseg, np.float64)
    _load().mmv_oracle_seg_sum_csr_f64(_p(x), _p(off), ctypes.c_int64(nseg), _p(out), _p(a))
    return out, a


def seg_sum_flags_bf16(xbits, f):
    x, fb = bf16_to_double(xbits), _as(f, np.uint8)
    n = x.shape[0]
    out, a = np.empty(max(n, 1), np.float64), np.empty(max(n, 1), np.float64)
    lib = _load()
    lib.mmv_oracle_seg_sum_flags_f64.restype = ctypes.c_int64
    k = lib.mmv_oracle_seg_sum_flags_f64(_p(x), _p(fb), ctypes.c_int64(n), _p(out), _p(a))
    return out[:k].copy(), a[:k].copy()


def seg_scan_excl_i8(x, f):
    """Segmented exclusive scan on int8 values, int32 result (low 32 bits of the exact sum)."""
    xb, fb = _as(x, np.int8), _as(f, np.uint8)
    n = xb.shape[0]
    assert fb.shape[0] == n
    e = np.empty(n, np.int32)
    _load().mmv_oracle_seg_scan_excl_i8(_p(xb), _p(fb), ctypes.c_int64(n), _p(e))
    return e


def flags_from_offsets(off, n):
    """f(i) = 1 iff i starts a non-empty segment of the CSR offsets ``off``."""
    off = _as(off, np.int32)
    nseg = off.shape[0] - 1
    f = np.empty(n, np.uint8)
    rc = _load().mmv_oracle_flags_from_offsets(_p(off), ctypes.c_int64(nseg), ctypes.c_int64(n), _p(f))
    if rc != 0:
        raise ValueError("offsets are not a non-decreasing sequence from 0 to n")
    return f


def seg_sum_flags_f16(x, f):
    xb, fb = _as_f16_bits(x), _as(f, np.uint8)
    n = xb.shape[0]
    out = np.empty(n, np.float64)
    a = np.empty(n, np.float64)
    k = _load().mmv_oracle_seg_sum_flags_f16(_p(xb), _p(fb), ctypes.c_int64(n), _p(out), _p(a))
    return out[:k].copy(), a[:k].copy()


def seg_sum_flags_i8(x, f):
    xb, fb = _as(x, np.int8), _as(f, np.uint8)
    n = xb.shape[0]
    out = np.empty(n, np.int32)
    k = _load().mmv_oracle_seg_sum_flags_i8(_p(xb), _p(fb), ctypes.c_int64(n), _p(out))
    return out[:k].copy()


def _check_offsets(off, n):
    if off.shape[0] < 1:
        raise ValueError("offsets need at least one entry")
    if off.shape[0] > 1:
        d = np.diff(off.astype(np.int64))
        if (d < 0).any():
            raise ValueError("offsets must be non-decreasing")
    if off[0] < 0 or off[-1] > n:
        raise ValueError("offsets out of range")


def seg_sum_csr_f16(x, off):
    xb, off = _as_f16_bits(x), _as(off, np.int32)
    _check_offsets(off, xb.shape[0])
    nseg = off.shape[0] - 1
    out = np.empty(nseg, np.float64)
    a = np.empty(nseg, np.float64)
    _load().mmv_oracle_seg_sum_csr_f16(_p(xb), _p(off), ctypes.c_int64(nseg), _p(out), _p(a))
    return out, a


def seg_sum_csr_i8(x, off):
    xb, off = _as(x, np.int8), _as(off, np.int32)
    _check_offsets(off, xb.shape[0])
    nseg = off.shape[0] - 1
    out = np.empty(nseg, np.int32)
    _load().mmv_oracle_seg_sum_csr_i8(_p(xb), _p(off), ctypes.c_int64(nseg), _p(out))
    return out


def spmv_csr(rowptr, col, val, x):
    rowptr, col = _as(rowptr, np.int32), _as(col, np.int32)
    vb, x = _as_f16_bits(val), _as(x, np.float32)
    _check_offsets(rowptr, vb.shape[0])
    if col.shape[0] and (col.min() < 0 or col.max() >= x.shape[0]):
        raise ValueError("column index out of range")
    rows = rowptr.shape[0] - 1
    y = np.empty(rows, np.float64)
    a = np.empty(rows, np.float64)
    _load().mmv_oracle_spmv_csr(_p(rowptr), _p(col), _p(vb), _p(x), ctypes.c_int64(rows), _p(y), _p(a))
    return y, a


def mult_i8(x, y) -> np.ndarray:
    """Element-wise product of two int8 vectors as int32 (Corollary 4.5)."""
    xb, yb = _as(x, np.int8), _as(y, np.int8)
    n = xb.shape[0]
    assert yb.shape[0] == n
    z = np.empty(n, np.int32)
    _load().mmv_oracle_mult_i8(_p(xb), _p(yb), ctypes.c_int64(n), _p(z))
    return z


def fp_bound(a):
    """Per-element error allowance of the fp16 -> fp32 paths."""
    return TOL_REL * np.asarray(a, np.float64) + TOL_ABS


def check_fp(got, z, a):
    """Compare an fp32 result with the oracle.  Returns (ok, worst_ratio, worst_index)."""
    got = np.asarray(got, np.float64)
    err = np.abs(got - z)
    bound = fp_bound(a)
    ratio = err / bound
    if ratio.size == 0:
        return True, 0.0, -1
    bad = ~np.isfinite(ratio)
    ratio = np.where(bad, np.inf, ratio)
    i = int(np.argmax(ratio))
    return bool(ratio[i] <= 1.0), float(ratio[i]), i
