"""Python binding of libmmv.so, the C-ABI CUDA library for segmented scan,
segmented sum and CSR SpMV on B200 (sm_100a).

The binding only marshals arguments: torch supplies device memory and the
current CUDA stream, every step of the computation runs in the library's own
kernels.  There is no CPU or PyTorch fallback: if the shared library is missing
the import of this module fails.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libmmv.so"

# enums of include/mmv.h
MMV_OK = 0
F16_TO_F32, I8_TO_I32, BF16_TO_F32 = 0, 1, 2
SEG_FLAGS_U8, SEG_OFFSETS_I32 = 0, 1
OP_SEG_SCAN, OP_SEG_SUM, OP_SPMV_CSR, OP_COMPRESS, OP_SEG_SCAN_MINMAX, OP_SEG_SCAN_WIDE, OP_MULT = 0, 1, 2, 3, 4, 5, 6

EXPORTS = (
    "mmv_workspace_bytes", "mmv_seg_scan", "mmv_seg_sum", "mmv_spmv_csr",
    "mmv_last_async_status", "mmv_status_string", "mmv_kernel_launch_count", "mmv_debug_configure",
    "mmv_seg_scan_static", "mmv_seg_scan_static_last_status", "mmv_debug_force_sum_groups",
    "mmv_seg_scan_host", "mmv_seg_scan_host_scratch_bytes", "mmv_seg_scan_exclusive", "mmv_compress",
    "mmv_seg_scan_minmax", "mmv_seg_scan_i8_i64", "mmv_seg_scan_shard", "mmv_seg_scan_shard_finish",
    "mmv_debug_force_scan_shape", "mmv_mult_i8",
)
SHARD_SUMMARY_BYTES = 16
STATIC_SCAN_MAX_N = 1 << 28


class MmvError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (mmv_status {code})")


def _load() -> ctypes.CDLL:
    if not LIB_PATH.exists():
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python paper_2506_23906_b200/build.py` "
            "(nvcc, sm_100a).  There is no fallback path.")
    lib = ctypes.CDLL(str(LIB_PATH))
    vp, i64, sz, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t, ctypes.c_int
    lib.mmv_workspace_bytes.restype = sz
    lib.mmv_workspace_bytes.argtypes = [ci, ci, ci, i64, i64]
    lib.mmv_seg_scan.restype = ci
    lib.mmv_seg_scan.argtypes = [vp, vp, ci, i64, i64, ci, vp, vp, sz, vp]
    lib.mmv_seg_scan_exclusive.restype = ci
    lib.mmv_seg_scan_exclusive.argtypes = [vp, vp, ci, i64, i64, ci, vp, vp, sz, vp]
    lib.mmv_seg_scan_minmax.restype = ci
    lib.mmv_seg_scan_minmax.argtypes = [vp, vp, i64, ci, ci, vp, vp, sz, vp]
    lib.mmv_seg_scan_i8_i64.restype = ci
    lib.mmv_seg_scan_i8_i64.argtypes = [vp, vp, i64, vp, vp, sz, vp]
    lib.mmv_compress.restype = ci
    lib.mmv_compress.argtypes = [vp, vp, i64, ci, vp, vp, vp, sz, vp]
    lib.mmv_seg_sum.restype = ci
    lib.mmv_seg_sum.argtypes = [vp, vp, ci, i64, i64, ci, vp, vp, vp, sz, vp]
    lib.mmv_spmv_csr.restype = ci
    lib.mmv_spmv_csr.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, vp, sz, vp]
    lib.mmv_last_async_status.restype = ci
    lib.mmv_last_async_status.argtypes = [vp, vp]
    lib.mmv_status_string.restype = ctypes.c_char_p
    lib.mmv_status_string.argtypes = [ci]
    lib.mmv_kernel_launch_count.restype = i64
    lib.mmv_kernel_launch_count.argtypes = []
    lib.mmv_seg_scan_static.restype = ci
    lib.mmv_seg_scan_static.argtypes = [vp, vp, i64, ci, vp, vp]
    lib.mmv_seg_scan_static_last_status.restype = ci
    lib.mmv_seg_scan_static_last_status.argtypes = [vp]
    lib.mmv_debug_configure.restype = None
    lib.mmv_debug_configure.argtypes = [i64, i64]
    lib.mmv_seg_scan_host_scratch_bytes.restype = sz
    lib.mmv_seg_scan_host_scratch_bytes.argtypes = [ci, i64]
    lib.mmv_seg_scan_host.restype = ci
    lib.mmv_seg_scan_host.argtypes = [vp, vp, i64, ci, vp, i64, vp, sz, vp]
    lib.mmv_seg_scan_shard.restype = ci
    lib.mmv_seg_scan_shard.argtypes = [vp, vp, i64, ci, ci, vp, vp, vp, sz, vp]
    lib.mmv_seg_scan_shard_finish.restype = ci
    lib.mmv_seg_scan_shard_finish.argtypes = [vp, ci, ci, vp, i64, ci, vp]
    lib.mmv_mult_i8.restype = ci
    lib.mmv_mult_i8.argtypes = [vp, vp, i64, vp, vp, sz, vp]
    lib.mmv_debug_force_scan_shape.restype = None
    lib.mmv_debug_force_scan_shape.argtypes = [ci]
    lib.mmv_debug_force_sum_groups.restype = None
    lib.mmv_debug_force_sum_groups.argtypes = [ci]
    return lib


_lib = _load()


def status_string(code: int) -> str:
    return _lib.mmv_status_string(int(code)).decode()


def kernel_launch_count() -> int:
    return int(_lib.mmv_kernel_launch_count())


def debug_configure(wait_budget_ns: int = 0, skip_publish_span: int = -1) -> None:
    _lib.mmv_debug_configure(int(wait_budget_ns), int(skip_publish_span))


def debug_force_scan_shape(shape: int = -1) -> None:
    _lib.mmv_debug_force_scan_shape(int(shape))


def debug_force_sum_groups(groups: int = 0) -> None:
    _lib.mmv_debug_force_sum_groups(int(groups))


def workspace_bytes(op: int, dt: int, sf: int, n: int, nseg: int = 0) -> int:
    return int(_lib.mmv_workspace_bytes(op, dt, sf, int(n), int(nseg)))


# (torch.cuda.current_stream() builds a Stream object, 5.7 us per call -- more than a small scan takes on the device;
#  the raw handle of the current stream comes back in a fraction of a microsecond where torch offers it)
_raw_current_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream_ptr(stream) -> int:
    if stream is not None:
        return int(stream.cuda_stream)
    if _raw_current_stream is not None:
        return int(_raw_current_stream(torch.cuda.current_device()))
    return int(torch.cuda.current_stream().cuda_stream)


def _ptr(t) -> int:
    return 0 if t is None else int(t.data_ptr())


def _dtype_code(x: torch.Tensor) -> int:
    if x.dtype == torch.float16:
        return F16_TO_F32
    if x.dtype == torch.int8:
        return I8_TO_I32
    if x.dtype == torch.bfloat16:
        return BF16_TO_F32
    raise TypeError("values must be torch.float16, torch.bfloat16 or torch.int8")


def _seg_code(seg: torch.Tensor) -> int:
    if seg.dtype == torch.uint8:
        return SEG_FLAGS_U8
    if seg.dtype == torch.int32:
        return SEG_OFFSETS_I32
    raise TypeError("segments must be uint8 start flags or int32 offsets")


def _check_cuda(*ts):
    for t in ts:
        if t is not None and (not t.is_cuda or not t.is_contiguous()):
            raise ValueError("tensors must be contiguous CUDA tensors")


def alloc_workspace(op: int, dt: int, sf: int, n: int, nseg: int = 0, device=None) -> torch.Tensor:
    nbytes = max(256, workspace_bytes(op, dt, sf, n, nseg))
    return torch.empty(nbytes, dtype=torch.uint8, device=device or "cuda")


def last_async_status(workspace: torch.Tensor, stream=None) -> int:
    return int(_lib.mmv_last_async_status(_ptr(workspace), _stream_ptr(stream)))


def seg_scan(x: torch.Tensor, seg: torch.Tensor | None, out: torch.Tensor | None = None,
             workspace: torch.Tensor | None = None, stream=None, exclusive: bool = False) -> torch.Tensor:
    """mmv_seg_scan: segmented inclusive scan (Problem 2.1, Eq. 1) of x over seg; seg = None is the
    plain inclusive scan (one segment, no flag vector is read).  exclusive=True calls
    mmv_seg_scan_exclusive: each element gets the sum of its segment's elements in front of it."""
    _check_cuda(x, seg, out, workspace)
    dt, sf = _dtype_code(x), (SEG_FLAGS_U8 if seg is None else _seg_code(seg))
    n = x.numel()
    nseg = seg.numel() - 1 if sf == SEG_OFFSETS_I32 else 0
    if out is None:
        out = torch.empty(n, dtype=torch.int32 if dt == I8_TO_I32 else torch.float32, device=x.device)
    if workspace is None:
        workspace = alloc_workspace(OP_SEG_SCAN, dt, sf, n, nseg, x.device)
    call = _lib.mmv_seg_scan_exclusive if exclusive else _lib.mmv_seg_scan
    rc = call(_ptr(x), _ptr(seg), sf, n, nseg, dt, _ptr(out), _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    if rc != MMV_OK:
        raise MmvError(rc, "mmv_seg_scan_exclusive" if exclusive else "mmv_seg_scan")
    return out


def seg_scan_shard(x: torch.Tensor, flags: torch.Tensor | None, first_shard: bool, out: torch.Tensor, summary: torch.Tensor,
                   workspace: torch.Tensor, stream=None) -> torch.Tensor:
    """mmv_seg_scan_shard: scan of one contiguous shard of a longer vector, without the carry from the shards in
    front of it; `summary` (16 bytes on the device, e.g. two int64) receives the shard's record."""
    _check_cuda(x, flags, out, summary, workspace)
    if summary.numel() * summary.element_size() < SHARD_SUMMARY_BYTES:
        raise ValueError("summary needs 16 bytes")
    rc = _lib.mmv_seg_scan_shard(_ptr(x), _ptr(flags), x.numel(), _dtype_code(x), 1 if first_shard else 0, _ptr(out),
                                 _ptr(summary), _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    if rc != MMV_OK:
        raise MmvError(rc, "mmv_seg_scan_shard")
    return out


def seg_scan_shard_finish(summaries: torch.Tensor, rank: int, world: int, out: torch.Tensor, x_dtype: torch.dtype,
                          stream=None) -> torch.Tensor:
    """mmv_seg_scan_shard_finish: fold the gathered records of the shards in front of `rank` and add the carry to
    this shard's elements in front of its first start."""
    _check_cuda(summaries, out)
    if summaries.numel() * summaries.element_size() < world * SHARD_SUMMARY_BYTES:
        raise ValueError("summaries needs 16 bytes per shard")
    dt = I8_TO_I32 if x_dtype == torch.int8 else (BF16_TO_F32 if x_dtype == torch.bfloat16 else F16_TO_F32)
    rc = _lib.mmv_seg_scan_shard_finish(_ptr(summaries), int(rank), int(world), _ptr(out), out.numel(), dt, _stream_ptr(stream))
    if rc != MMV_OK:
        raise MmvError(rc, "mmv_seg_scan_shard_finish")
    return out


def mult_i8(x: torch.Tensor, y: torch.Tensor, out: torch.Tensor | None = None, workspace: torch.Tensor | None = None,
            stream=None) -> torch.Tensor:
    """mmv_mult_i8: element-wise product of two int8 vectors through the segmented sum (Corollary 4.5), int32."""
    _check_cuda(x, y, out, workspace)
    if x.dtype != torch.int8 or y.dtype != torch.int8 or x.numel() != y.numel():
        raise TypeError("two int8 vectors of the same length expected")
    n = x.numel()
    if out is None:
        out = torch.empty(n, dtype=torch.int32, device=x.device)
    if workspace is None:
        workspace = alloc_workspace(OP_MULT, I8_TO_I32, SEG_OFFSETS_I32, n, 0, x.device)
    rc = _lib.mmv_mult_i8(_ptr(x), _ptr(y), n, _ptr(out), _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    if rc != MMV_OK:
        raise MmvError(rc, "mmv_mult_i8")
    return out


def seg_scan_minmax(x: torch.Tensor, flags: torch.Tensor | None, want_min: bool = False, out: torch.Tensor | None = None,
                    workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """mmv_seg_scan_minmax: segmented running maximum (or minimum) of fp16 / int8 values; flags = None is one segment."""
    _check_cuda(x, flags, out, workspace)
    dt, n = _dtype_code(x), x.numel()
    if out is None:
        out = torch.empty(n, dtype=torch.int32 if dt == I8_TO_I32 else torch.float32, device=x.device)
    if workspace is None:
        workspace = alloc_workspace(OP_SEG_SCAN_MINMAX, dt, SEG_FLAGS_U8, n, 0, x.device)
    rc = _lib.mmv_seg_scan_minmax(_ptr(x), _ptr(flags), n, dt, int(bool(want_min)), _ptr(out), _ptr(workspace),
                                  workspace.numel(), _stream_ptr(stream))
    if rc != MMV_OK:
        raise MmvError(rc, "mmv_seg_scan_minmax")
    return out


def seg_scan_wide(x: torch.Tensor, flags: torch.Tensor | None, out: torch.Tensor | None = None,
                  workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """mmv_seg_scan_i8_i64: segmented inclusive scan of int8 values with int64 results (no wrap); flags = None is one segment."""
    _check_cuda(x, flags, out, workspace)
    if x.dtype != torch.int8:
        raise TypeError("seg_scan_wide takes int8 values")
    n = x.numel()
    if out is None:
        out = torch.empty(n, dtype=torch.int64, device=x.device)
    if workspace is None:
        workspace = alloc_workspace(OP_SEG_SCAN_WIDE, I8_TO_I32, SEG_FLAGS_U8, n, 0, x.device)
    rc = _lib.mmv_seg_scan_i8_i64(_ptr(x), _ptr(flags), n, _ptr(out), _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    if rc != MMV_OK:
        raise MmvError(rc, "mmv_seg_scan_i8_i64")
    return out


def compress(x: torch.Tensor, flags: torch.Tensor, out: torch.Tensor | None = None, count: torch.Tensor | None = None,
             workspace: torch.Tensor | None = None, stream=None):
    """mmv_compress: COMPRESS of Section 2 -- the values x[i] with flags[i] != 0, in order.  Returns (out, count):
    out has room for n values of x's type, count is an int64 device tensor holding K; out[:K] is the result."""
    _check_cuda(x, flags, out, workspace)
    if flags.dtype != torch.uint8:
        raise TypeError("flags must be uint8")
    dt, n = _dtype_code(x), x.numel()
    if out is None:
        out = torch.empty(n, dtype=x.dtype, device=x.device)
    if count is None:
        count = torch.zeros(1, dtype=torch.int64, device=x.device)
    if workspace is None:
        workspace = alloc_workspace(OP_COMPRESS, dt, SEG_FLAGS_U8, n, 0, x.device)
    rc = _lib.mmv_compress(_ptr(x), _ptr(flags), n, dt, _ptr(out), _ptr(count), _ptr(workspace), workspace.numel(),
                           _stream_ptr(stream))
    if rc != MMV_OK:
        raise MmvError(rc, "mmv_compress")
    return out, count


def seg_scan_static(x: torch.Tensor, flags: torch.Tensor, out: torch.Tensor, stream=None) -> torch.Tensor:
    """mmv_seg_scan_static: the scan for callers that can pass only inputs and outputs.

    The carry words live in a buffer built into the library, so nothing is allocated by the
    call (here the caller supplies ``out`` too).  n is limited to STATIC_SCAN_MAX_N; calls on
    one device must not overlap on the GPU.
    """
    _check_cuda(x, flags, out)
    if flags.dtype != torch.uint8:
        raise TypeError("start flags must be uint8")
    rc = _lib.mmv_seg_scan_static(_ptr(x), _ptr(flags), x.numel(), _dtype_code(x), _ptr(out), _stream_ptr(stream))
    if rc != MMV_OK:
        raise MmvError(rc, "mmv_seg_scan_static")
    return out


def host_scan_scratch(dt: int, chunk: int, device=None) -> torch.Tensor:
    nbytes = int(_lib.mmv_seg_scan_host_scratch_bytes(dt, int(chunk)))
    if nbytes == 0:
        raise ValueError("chunk must be a positive multiple of 16384")
    return torch.empty(nbytes, dtype=torch.uint8, device=device or "cuda")


def seg_scan_host(x: torch.Tensor, flags: torch.Tensor | None, out: torch.Tensor | None = None, chunk: int = 1 << 26,
                  scratch: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """mmv_seg_scan_host: the scan of HOST tensors (pinned memory recommended), copies and kernels
    of neighbouring chunks overlapped.  Returns ``out`` (a pinned host tensor unless one is given);
    the results are complete once the stream has been synchronised."""
    if x.is_cuda or (flags is not None and flags.is_cuda) or (out is not None and out.is_cuda):
        raise ValueError("seg_scan_host takes host tensors")
    if not x.is_contiguous() or (flags is not None and (flags.dtype != torch.uint8 or not flags.is_contiguous())):
        raise TypeError("contiguous values and uint8 start flags expected")
    dt = _dtype_code(x)
    n = x.numel()
    if out is None:
        out = torch.empty(n, dtype=torch.int32 if dt == I8_TO_I32 else torch.float32, pin_memory=True)
    if scratch is None:
        scratch = host_scan_scratch(dt, chunk)
    rc = _lib.mmv_seg_scan_host(_ptr(x), _ptr(flags), n, dt, _ptr(out), int(chunk), _ptr(scratch), scratch.numel(),
                                _stream_ptr(stream))
    if rc != MMV_OK:
        raise MmvError(rc, "mmv_seg_scan_host")
    return out


def seg_scan_static_last_status(stream=None) -> int:
    return int(_lib.mmv_seg_scan_static_last_status(_stream_ptr(stream)))


def seg_sum(x: torch.Tensor, seg: torch.Tensor, out: torch.Tensor | None = None,
            num_segments: torch.Tensor | None = None, workspace: torch.Tensor | None = None,
            stream=None) -> torch.Tensor:
    """mmv_seg_sum: per-segment sums (Section 2) of x over seg (CSR offsets or flags)."""
    _check_cuda(x, seg, out, workspace, num_segments)
    dt, sf = _dtype_code(x), _seg_code(seg)
    n = x.numel()
    nseg = seg.numel() - 1 if sf == SEG_OFFSETS_I32 else 0
    if out is None:
        cap = nseg if sf == SEG_OFFSETS_I32 else n
        out = torch.empty(cap, dtype=torch.int32 if dt == I8_TO_I32 else torch.float32, device=x.device)
    if workspace is None:
        workspace = alloc_workspace(OP_SEG_SUM, dt, sf, n, nseg, x.device)
    rc = _lib.mmv_seg_sum(_ptr(x), _ptr(seg), sf, n, nseg, dt, _ptr(out), _ptr(num_segments),
                          _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    if rc != MMV_OK:
        raise MmvError(rc, "mmv_seg_sum")
    return out


def spmv_csr(rowptr: torch.Tensor, col: torch.Tensor, val: torch.Tensor, x: torch.Tensor,
             y: torch.Tensor | None = None, workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """mmv_spmv_csr: y = A x for a CSR matrix (Algorithm 4.4), fp16 values, fp32 x and y."""
    _check_cuda(rowptr, col, val, x, y, workspace)
    if rowptr.dtype != torch.int32 or col.dtype != torch.int32 or val.dtype != torch.float16 or x.dtype != torch.float32:
        raise TypeError("rowptr/col int32, val float16, x float32 expected")
    rows, cols, nnz = rowptr.numel() - 1, x.numel(), val.numel()
    if y is None:
        y = torch.empty(rows, dtype=torch.float32, device=x.device)
    if workspace is None:
        workspace = alloc_workspace(OP_SPMV_CSR, F16_TO_F32, SEG_OFFSETS_I32, nnz, rows, x.device)
    rc = _lib.mmv_spmv_csr(_ptr(rowptr), _ptr(col), _ptr(val), _ptr(x), _ptr(y), rows, cols, nnz,
                           _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    if rc != MMV_OK:
        raise MmvError(rc, "mmv_spmv_csr")
    return y
