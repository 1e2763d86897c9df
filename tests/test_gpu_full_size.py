"""Parity at the sizes and in the launch configuration that bench.py times.

The same binding calls as the benchmark (device-resident inputs, one workspace, current stream),
on the full-size synthetic workloads; the oracle is streamed over the arrays chunk by chunk (it
keeps its running state between chunks), so that no more than a chunk of fp64 reference values is
ever held.
"""
import numpy as np
import pytest

import mmv_inputs as gen
import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

STEP = 1 << 24


@pytest.fixture(scope="module")
def mmv():
    if not torch.cuda.is_available():
        pytest.skip("no GPU")
    import paper_2506_23906_b200 as m
    return m


def stream_check_f16(x, f, out_d, what, lo=0, hi=None, state=None):
    """Oracle streamed over [lo, hi) with carried state; returns the largest |error| / bound."""
    hi = x.shape[0] if hi is None else hi
    state = oracle.new_f16_state() if state is None else state
    worst = 0.0
    for o in range(lo, hi, STEP):
        e = min(hi, o + STEP)
        z, a = oracle.seg_scan_f16(x[o:e], f[o:e], state)
        ok, ratio, i = oracle.check_fp(out_d[o:e].cpu().numpy(), z, a)
        assert ok, f"{what}: outside the bound at element {o + i} (ratio {ratio})"
        worst = max(worst, ratio)
    return worst


@pytest.fixture(scope="module")
def c5_values():
    return gen.config5_values(1 << 30)


@pytest.mark.parametrize("case", [c for c, _ in gen.C5_CASES])
def test_config5_full_size(mmv, c5_values, case):
    x = c5_values
    n = x.shape[0]
    f = gen.config5_flags(n, case)
    xd, fd = torch.from_numpy(x).cuda(), torch.from_numpy(f).cuda()
    od = torch.empty(n, dtype=torch.float32, device="cuda")
    ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN, mmv.F16_TO_F32, mmv.SEG_FLAGS_U8, n)
    for _ in range(2):                                   # as in the benchmark: repeated launches, one workspace
        mmv.seg_scan(xd, fd, out=od, workspace=ws)
    assert mmv.last_async_status(ws) == 0
    # every one of the 2^30 elements, for all seven flag patterns (the oracle streams with carried state)
    stream_check_f16(x, f, od, f"config 5 / {case}")
    del xd, fd, od, ws
    torch.cuda.empty_cache()


def test_config3_full_size(mmv):
    x, f = gen.config3()
    n = x.shape[0]
    xd, fd = torch.from_numpy(x).cuda(), torch.from_numpy(f).cuda()
    od = torch.empty(n, dtype=torch.int32, device="cuda")
    ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN, mmv.I8_TO_I32, mmv.SEG_FLAGS_U8, n)
    mmv.seg_scan(xd, fd, out=od, workspace=ws)
    assert mmv.last_async_status(ws) == 0
    state = oracle.new_i8_state()
    for o in range(0, n, STEP):
        want = oracle.seg_scan_i8(x[o:o + STEP], f[o:o + STEP], state)
        assert np.array_equal(od[o:o + STEP].cpu().numpy(), want), f"config 3: mismatch in chunk at {o}"


def test_config2_full_size_and_four_times_larger_with_both_encodings(mmv):
    for n in (1 << 26, 1 << 28):
        x, off = gen.config2(n)
        nseg = off.shape[0] - 1
        want, a = oracle.seg_sum_csr_f16(x, off)
        xd = torch.from_numpy(x).cuda()
        ws = mmv.alloc_workspace(mmv.OP_SEG_SUM, mmv.F16_TO_F32, mmv.SEG_OFFSETS_I32, n, nseg)
        out = mmv.seg_sum(xd, torch.from_numpy(off).cuda(), workspace=ws)
        assert mmv.last_async_status(ws) == 0
        ok, ratio, i = oracle.check_fp(out.cpu().numpy(), want, a)
        assert ok, f"config 2 (n = {n}): ratio {ratio} at segment {i}"
        if n == 1 << 28:
            f = gen.start_flags_of_offsets(off, n)
            wantf, af = oracle.seg_sum_flags_f16(x, f)
            ws = mmv.alloc_workspace(mmv.OP_SEG_SUM, mmv.F16_TO_F32, mmv.SEG_FLAGS_U8, n)
            kd = torch.zeros(1, dtype=torch.int64, device="cuda")
            outf = mmv.seg_sum(xd, torch.from_numpy(f).cuda(), num_segments=kd, workspace=ws)
            assert mmv.last_async_status(ws) == 0
            assert int(kd.item()) == wantf.shape[0]
            ok, ratio, i = oracle.check_fp(outf[:wantf.shape[0]].cpu().numpy(), wantf, af)
            assert ok, f"flag-encoded config 2 (n = {n}): ratio {ratio} at segment {i}"
        del xd, ws
        torch.cuda.empty_cache()


@pytest.mark.parametrize("empty_fraction", [0.0, 0.1])
def test_config4_full_size(mmv, empty_fraction):
    rowptr, col, val, xv = gen.config4(empty_fraction=empty_fraction)
    rows = rowptr.shape[0] - 1
    ws = mmv.alloc_workspace(mmv.OP_SPMV_CSR, mmv.F16_TO_F32, mmv.SEG_OFFSETS_I32, val.shape[0], rows)
    y = mmv.spmv_csr(torch.from_numpy(rowptr).cuda(), torch.from_numpy(col).cuda(), torch.from_numpy(val).cuda(),
                     torch.from_numpy(xv).cuda(), workspace=ws)
    assert mmv.last_async_status(ws) == 0
    want, a = oracle.spmv_csr(rowptr, col, val, xv)
    ok, ratio, i = oracle.check_fp(y.cpu().numpy(), want, a)
    assert ok, f"config 4 (empty rows {empty_fraction}): ratio {ratio} at row {i}"
    if empty_fraction:
        lens = np.diff(rowptr.astype(np.int64))
        assert (y.cpu().numpy()[lens == 0] == 0).all()


def test_block_sparse_attention_full_size(mmv):
    # the largest of the blocked sparse-attention matrices at the paper's size: 65,536 rows, b-64_r-8
    rowptr, col, val, xv = gen.block_sparse_attention_csr(64, 8)
    rows, nnz = rowptr.shape[0] - 1, val.shape[0]
    rd, cd, vd, xd = (torch.from_numpy(t).cuda() for t in (rowptr, col, val, xv))
    ws = mmv.alloc_workspace(mmv.OP_SPMV_CSR, mmv.F16_TO_F32, mmv.SEG_OFFSETS_I32, nnz, rows)
    y = mmv.spmv_csr(rd, cd, vd, xd, workspace=ws)
    assert mmv.last_async_status(ws) == 0
    want, a = oracle.spmv_csr(rowptr, col, val, xv)
    ok, ratio, i = oracle.check_fp(y.cpu().numpy(), want, a)
    assert ok, f"b-64_r-8: |err|/bound = {ratio:.3g} at row {i}"


@pytest.mark.parametrize("kind", gen.ROW_LENGTH_MIXES)
def test_row_length_mixes_at_bench_size(mmv, kind):
    x, off = gen.seg_sum_row_mix(kind, 1 << 26)
    nseg = off.shape[0] - 1
    xd, od = torch.from_numpy(x).cuda(), torch.from_numpy(off).cuda()
    ws = mmv.alloc_workspace(mmv.OP_SEG_SUM, mmv.F16_TO_F32, mmv.SEG_OFFSETS_I32, x.shape[0], nseg)
    got = mmv.seg_sum(xd, od, workspace=ws)
    assert mmv.last_async_status(ws) == 0
    want, a = oracle.seg_sum_csr_f16(x, off)
    ok, ratio, i = oracle.check_fp(got.cpu().numpy(), want, a)
    assert ok, f"{kind}: |err|/bound = {ratio:.3g} at segment {i}"


@pytest.mark.parametrize("seglen", [1000, 3_000_001])
def test_seg_sum_just_below_2_to_the_31_elements_closed_form(mmv, seglen):
    """The largest input the offset encoding admits (positions are 32-bit): all-ones int8 values in segments of a
    constant length that is no divisor of the span size, short ones (general path) and long ones (few-boundaries
    path, carries across thousands of spans); every sum is the segment's length."""
    n = (1 << 31) - 16
    free, _ = torch.cuda.mem_get_info()
    if free < n + (1 << 30):
        pytest.skip("not enough device memory")
    x = torch.ones(n, dtype=torch.int8, device="cuda")
    nseg = (n + seglen - 1) // seglen
    off = torch.arange(nseg + 1, dtype=torch.int64, device="cuda") * seglen
    off[-1] = n
    off = off.to(torch.int32)
    ws = mmv.alloc_workspace(mmv.OP_SEG_SUM, mmv.I8_TO_I32, mmv.SEG_OFFSETS_I32, n, nseg)
    out = mmv.seg_sum(x, off, workspace=ws)
    assert mmv.last_async_status(ws) == 0
    want = torch.full((nseg,), seglen, dtype=torch.int32, device="cuda")
    want[-1] = n - seglen * (nseg - 1)
    assert torch.equal(out, want)
    del x, off, out, ws
    torch.cuda.empty_cache()


def test_spmv_just_below_2_to_the_31_products_closed_form(mmv):
    """The largest matrix the 32-bit row pointers admit: every value 1, x = 1, rows of 777 products (the last one
    shorter), columns spread over x; y(r) = length of row r, exactly (sums of ones below 2^24)."""
    nnz = (1 << 31) - 16
    free, _ = torch.cuda.mem_get_info()
    if free < 12 * nnz + (2 << 30):
        pytest.skip("not enough device memory")
    rowlen, cols = 777, 1 << 20
    rows = (nnz + rowlen - 1) // rowlen
    rowptr = torch.arange(rows + 1, dtype=torch.int64, device="cuda") * rowlen
    rowptr[-1] = nnz
    rowptr = rowptr.to(torch.int32)
    col = torch.empty(nnz, dtype=torch.int32, device="cuda")
    step = 1 << 28
    for o in range(0, nnz, step):
        e = min(nnz, o + step)
        col[o:e] = ((torch.arange(o, e, dtype=torch.int64, device="cuda") * 2654435761) % cols).to(torch.int32)
    val = torch.ones(nnz, dtype=torch.float16, device="cuda")
    xv = torch.ones(cols, dtype=torch.float32, device="cuda")
    ws = mmv.alloc_workspace(mmv.OP_SPMV_CSR, mmv.F16_TO_F32, mmv.SEG_OFFSETS_I32, nnz, rows)
    y = mmv.spmv_csr(rowptr, col, val, xv, workspace=ws)
    assert mmv.last_async_status(ws) == 0
    want = torch.full((rows,), float(rowlen), dtype=torch.float32, device="cuda")
    want[-1] = float(nnz - rowlen * (rows - 1))
    assert torch.equal(y, want)
    del rowptr, col, val, xv, ws, y
    torch.cuda.empty_cache()


@pytest.mark.parametrize("period", [1, 3, 1000])
def test_compress_just_below_2_to_the_31_elements_closed_form(mmv, period):
    """COMPRESS at its largest size: x(i) = (i mod 251) - 125, every period-th element kept (all of them, a
    third: the staged route; one in a thousand: the sparse loop), so kept(j) = x(period * j)."""
    n = (1 << 31) - 16
    free, _ = torch.cuda.mem_get_info()
    if free < 4 * n + (2 << 30):
        pytest.skip("not enough device memory")
    x = torch.empty(n, dtype=torch.int8, device="cuda")
    f = torch.zeros(n, dtype=torch.uint8, device="cuda")
    step = 1 << 28
    for o in range(0, n, step):
        e = min(n, o + step)
        idx = torch.arange(o, e, dtype=torch.int64, device="cuda")
        x[o:e] = (idx % 251 - 125).to(torch.int8)
        f[o:e] = (idx % period == 0).to(torch.uint8) * 7
        del idx
    ws = mmv.alloc_workspace(mmv.OP_COMPRESS, mmv.I8_TO_I32, mmv.SEG_FLAGS_U8, n)
    out, count = mmv.compress(x, f, workspace=ws)
    assert mmv.last_async_status(ws) == 0
    k = (n + period - 1) // period
    assert int(count.item()) == k
    for o in range(0, k, step):
        e = min(k, o + step)
        j = torch.arange(o, e, dtype=torch.int64, device="cuda")
        assert torch.equal(out[o:e], ((j * period) % 251 - 125).to(torch.int8)), f"kept values wrong in [{o}, {e})"
        del j
    del x, f, out, ws
    torch.cuda.empty_cache()


def test_scan_beyond_2_to_the_32_elements_closed_form(mmv):
    """Index arithmetic past 2^32 elements: all-ones int8 values with a start flag every 1000 elements
    (one period is not a divisor of the tile size, so the flags drift through every position of a
    tile), for which the scan has the closed form z[i] = (i mod 1000) + 1; checked chunk by chunk on
    the device.  A second launch without flags is checked against z[i] = i + 1 modulo 2^32."""
    n = (1 << 32) + 12345
    free, _ = torch.cuda.mem_get_info()
    if free < 6 * n + (2 << 30):
        pytest.skip("not enough device memory for a 2^32-element scan")
    x = torch.ones(n, dtype=torch.int8, device="cuda")
    f = torch.zeros(n, dtype=torch.uint8, device="cuda")
    f[::1000] = 1
    out = torch.empty(n, dtype=torch.int32, device="cuda")
    ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN, mmv.I8_TO_I32, mmv.SEG_FLAGS_U8, n)
    mmv.seg_scan(x, f, out=out, workspace=ws)
    assert mmv.last_async_status(ws) == 0
    step = 1 << 27
    for o in range(0, n, step):
        e = min(n, o + step)
        idx = torch.arange(o, e, dtype=torch.int64, device="cuda")
        assert torch.equal(out[o:e], (idx % 1000 + 1).to(torch.int32)), f"flagged scan wrong in [{o}, {e})"
    del f
    mmv.seg_scan(x, None, out=out, workspace=ws)
    assert mmv.last_async_status(ws) == 0
    for o in range(0, n, step):
        e = min(n, o + step)
        idx = torch.arange(o + 1, e + 1, dtype=torch.int64, device="cuda")
        want = (idx & 0xffffffff).to(torch.int64)
        want = torch.where(want >= (1 << 31), want - (1 << 32), want).to(torch.int32)     # wrap-around modulo 2^32
        assert torch.equal(out[o:e], want), f"plain scan wrong in [{o}, {e})"


def test_exclusive_scan_full_size(mmv, c5_values):
    # the exclusive variant at the headline size: exclusive + element = inclusive, checked piecewise against the
    # oracle's inclusive scan streamed over the array
    n = 1 << 30
    f = gen.config5_flags(n, "p1e-3")
    xd, fd = torch.from_numpy(c5_values).cuda(), torch.from_numpy(f).cuda()
    ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN, mmv.F16_TO_F32, mmv.SEG_FLAGS_U8, n)
    out = mmv.seg_scan(xd, fd, workspace=ws, exclusive=True)
    assert mmv.last_async_status(ws) == 0
    state = oracle.new_f16_state()
    worst = 0.0
    for lo in range(0, n, STEP):
        hi = min(n, lo + STEP)
        z, a = oracle.seg_scan_f16(c5_values[lo:hi], f[lo:hi], state)
        xs = c5_values[lo:hi].astype(np.float64)
        want = z - xs                                           # exact in fp64 for these magnitudes
        bound = oracle.fp_bound(np.maximum(a - np.abs(xs), 0.0))       # sum of |x| over the elements in front
        got = out[lo:hi].cpu().numpy().astype(np.float64)
        worst = max(worst, float(np.max(np.abs(got - want) / bound)))
        starts = f[lo:hi] != 0
        assert (got[starts] == 0.0).all()
    assert worst <= 1.0, f"exclusive scan: |err|/bound = {worst}"


def test_running_maximum_full_size(mmv, c5_values):
    # the segmented running maximum at the headline size against the oracle, chunk by chunk: a chunk's elements in
    # front of its first start take the maximum with the value carried out of the chunk before
    n = 1 << 30
    f = gen.config5_flags(n, "p1e-3")
    xd, fd = torch.from_numpy(c5_values).cuda(), torch.from_numpy(f).cuda()
    ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN_MINMAX, mmv.F16_TO_F32, mmv.SEG_FLAGS_U8, n)
    out = mmv.seg_scan_minmax(xd, fd, workspace=ws)
    assert mmv.last_async_status(ws) == 0
    carry = -np.inf
    for lo in range(0, n, STEP):
        hi = min(n, lo + STEP)
        z = oracle.seg_scan_minmax_f16(c5_values[lo:hi], f[lo:hi])
        starts = np.flatnonzero(f[lo:hi])
        first = int(starts[0]) if starts.size else hi - lo
        z[:first] = np.maximum(z[:first], carry)
        carry = z[-1]
        assert np.array_equal(out[lo:hi].cpu().numpy().astype(np.float64), z), f"running maximum wrong in [{lo}, {hi})"
    # and without a flag vector: every element is the maximum of all elements up to it
    out = mmv.seg_scan_minmax(xd, None, workspace=ws)
    assert mmv.last_async_status(ws) == 0
    carry = -np.inf
    for lo in range(0, n, STEP):
        hi = min(n, lo + STEP)
        z = np.maximum(np.maximum.accumulate(c5_values[lo:hi].astype(np.float32)), np.float32(carry))
        carry = z[-1]
        assert np.array_equal(out[lo:hi].cpu().numpy(), z), f"plain running maximum wrong in [{lo}, {hi})"


def test_wide_integer_scan_full_size(mmv):
    # int8 -> int64 at 2^30 elements, flags p = 1e-3, against the oracle chunk by chunk: a chunk's elements in front
    # of its first start add the value carried out of the chunk before; then one segment of 2^30 values of -128,
    # whose sums pass the int32 range 64 times over (closed form)
    n = 1 << 30
    f = gen.config5_flags(n, "p1e-3")
    x = gen.i8_uniform(3, n)
    xd, fd = torch.from_numpy(x).cuda(), torch.from_numpy(f).cuda()
    ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN_WIDE, mmv.I8_TO_I32, mmv.SEG_FLAGS_U8, n)
    out = mmv.seg_scan_wide(xd, fd, workspace=ws)
    assert mmv.last_async_status(ws) == 0
    carry = 0
    for lo in range(0, n, STEP):
        hi = min(n, lo + STEP)
        z = oracle.seg_scan_i8_wide(x[lo:hi], f[lo:hi])
        starts = np.flatnonzero(f[lo:hi])
        first = int(starts[0]) if starts.size else hi - lo
        z[:first] += carry
        carry = int(z[-1])
        assert np.array_equal(out[lo:hi].cpu().numpy(), z), f"int64 scan wrong in [{lo}, {hi})"
    del xd, fd
    xd = torch.full((n,), -128, dtype=torch.int8, device="cuda")
    out = mmv.seg_scan_wide(xd, None, out=out, workspace=ws)
    assert mmv.last_async_status(ws) == 0
    for lo in range(0, n, STEP):
        hi = min(n, lo + STEP)
        want = torch.arange(lo + 1, hi + 1, dtype=torch.int64, device="cuda") * -128
        assert torch.equal(out[lo:hi], want), f"int64 plain scan wrong in [{lo}, {hi})"


@pytest.mark.parametrize("case", ["p1e-3", "p0.5"])
def test_compress_full_size(mmv, c5_values, case):
    # COMPRESS of the headline values under the headline flags (one in a thousand kept: every lane walks its own
    # mask) and under the flags with every second element kept (warps stage their kept values in shared
    # memory): the kept values are x[f != 0], in order
    n = 1 << 30
    f = gen.config5_flags(n, case)
    xd, fd = torch.from_numpy(c5_values).cuda(), torch.from_numpy(f).cuda()
    ws = mmv.alloc_workspace(mmv.OP_COMPRESS, mmv.F16_TO_F32, mmv.SEG_FLAGS_U8, n)
    out, count = mmv.compress(xd, fd, workspace=ws)
    assert mmv.last_async_status(ws) == 0
    k = int(count.item())
    pos = 0
    for lo in range(0, n, STEP):
        hi = min(n, lo + STEP)
        kept = oracle.compress(c5_values[lo:hi], f[lo:hi])
        got = out[pos:pos + kept.shape[0]].cpu().numpy()
        assert np.array_equal(got.view(np.uint16), kept.view(np.uint16)), f"COMPRESS wrong for the flags in [{lo}, {hi})"
        pos += kept.shape[0]
    assert pos == k


def test_bf16_scan_full_size(mmv, c5_values):
    # bfloat16 values (the headline values rounded to bf16 on the device) under the headline flags, against the
    # oracle chunk by chunk: the elements in front of a chunk's first start add what the chunk before carried out
    n = 1 << 30
    f = gen.config5_flags(n, "p1e-3")
    xb = torch.from_numpy(c5_values).cuda().to(torch.bfloat16)
    fd = torch.from_numpy(f).cuda()
    ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN, mmv.BF16_TO_F32, mmv.SEG_FLAGS_U8, n)
    out = mmv.seg_scan(xb, fd, workspace=ws)
    assert mmv.last_async_status(ws) == 0
    bits = xb.view(torch.int16)
    carry_z, carry_a, worst = 0.0, 0.0, 0.0
    for lo in range(0, n, STEP):
        hi = min(n, lo + STEP)
        z, a = oracle.seg_scan_bf16(bits[lo:hi].cpu().numpy().view(np.uint16), f[lo:hi])
        starts = np.flatnonzero(f[lo:hi])
        first = int(starts[0]) if starts.size else hi - lo
        if lo > 0:
            z[:first] += carry_z
            a[:first] += carry_a
        carry_z, carry_a = float(z[-1]), float(a[-1])
        ok, ratio, i = oracle.check_fp(out[lo:hi].cpu().numpy(), z, a)
        assert ok, f"bf16 scan: outside the bound at element {lo + i} (ratio {ratio})"
        worst = max(worst, ratio)
    assert worst <= 1.0
