"""Parity of the CUDA library (through its C ABI) with the CPU oracle.

int8 -> int32 paths are compared bit for bit; fp16 -> fp32 paths must satisfy
|gpu - oracle| <= 2e-3 * (sum of |x| over the summed range) + 1e-6 per element.
Sizes span several 16384-element tiles and ragged tails.
"""
import numpy as np
import pytest

import mmv_inputs as gen
import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TILE = 16384


@pytest.fixture(scope="module")
def mmv():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2506_23906_b200 as m
    m.debug_configure(0, -1)
    return m


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def scan_i8(mmv, x, f, guard=64, exclusive=False):
    n = x.shape[0]
    seg = dev(f)
    sf = mmv.SEG_FLAGS_U8 if f.dtype == np.uint8 else mmv.SEG_OFFSETS_I32
    ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN, mmv.I8_TO_I32, sf, n, max(0, f.shape[0] - 1))
    buf = torch.full((n + guard,), -777, dtype=torch.int32, device="cuda")
    mmv.seg_scan(dev(x), seg, out=buf[:n], workspace=ws, exclusive=exclusive)
    assert mmv.last_async_status(ws) == 0
    got = buf.cpu().numpy()
    assert (got[n:] == -777).all(), "wrote past the end of the output"
    return got[:n]


def scan_f16(mmv, x, f, guard=64, exclusive=False):
    n = x.shape[0]
    sf = mmv.SEG_FLAGS_U8 if f.dtype == np.uint8 else mmv.SEG_OFFSETS_I32
    ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN, mmv.F16_TO_F32, sf, n, max(0, f.shape[0] - 1))
    buf = torch.full((n + guard,), -777.0, dtype=torch.float32, device="cuda")
    mmv.seg_scan(dev(x), dev(f), out=buf[:n], workspace=ws, exclusive=exclusive)
    assert mmv.last_async_status(ws) == 0
    got = buf.cpu().numpy()
    assert (got[n:] == -777.0).all(), "wrote past the end of the output"
    return got[:n]


def assert_fp(got, z, a, what):
    ok, ratio, i = oracle.check_fp(got, z, a)
    assert ok, f"{what}: |err|/bound = {ratio:.3g} at index {i}: got {got[i]!r}, want {z[i]!r}"
    return ratio


SIZES = [1, 2, 31, 32, 33, 1023, 1024, 1025, 4095, 4096, 4097, TILE - 1, TILE, TILE + 1,
         2 * TILE - 1, 2 * TILE + 1, 5 * TILE + 4099, 100_003]


@pytest.mark.parametrize("n", SIZES)
def test_scan_i8_sizes(mmv, n):
    rng = np.random.default_rng(n)
    x = rng.integers(-128, 128, n).astype(np.int8)
    for p in (0.0, 0.01, 0.3, 1.0):
        f = (rng.random(n) < p).astype(np.uint8)
        assert np.array_equal(scan_i8(mmv, x, f), oracle.seg_scan_i8(x, f)), (n, p)


@pytest.mark.parametrize("n", SIZES)
def test_scan_f16_sizes(mmv, n):
    rng = np.random.default_rng(n + 1)
    x = rng.uniform(-1, 1, n).astype(np.float16)
    for p in (0.0, 1.0 / 64, 0.5, 1.0):
        f = (rng.random(n) < p).astype(np.uint8)
        z, a = oracle.seg_scan_f16(x, f)
        assert_fp(scan_f16(mmv, x, f), z, a, f"n={n} p={p}")


def test_scan_flag_positions_around_row_and_tile_edges(mmv):
    n = 3 * TILE
    rng = np.random.default_rng(5)
    x = rng.integers(-8, 8, n).astype(np.int8)
    xf = rng.uniform(-1, 1, n).astype(np.float16)
    for pos in (1, 31, 32, 33, 1023, 1024, 4095, 4096, 4097, TILE - 1, TILE, TILE + 1, 2 * TILE, n - 1):
        f = np.zeros(n, np.uint8)
        f[pos] = 1
        assert np.array_equal(scan_i8(mmv, x, f), oracle.seg_scan_i8(x, f)), pos
        f[min(n - 1, pos + 1)] = 1
        f[pos - 1] = 1
        assert np.array_equal(scan_i8(mmv, x, f), oracle.seg_scan_i8(x, f)), pos
        z, a = oracle.seg_scan_f16(xf, f)
        assert_fp(scan_f16(mmv, xf, f), z, a, f"flags around {pos}")


def test_scan_closed_forms(mmv):
    n = 2 * TILE + 77
    ones = np.ones(n, np.int8)
    f = gen.flags(9, n, pattern="cycle123")
    assert np.array_equal(scan_i8(mmv, ones, f), np.tile([1, 1, 2, 1, 2, 3], n // 6 + 1)[:n])
    f = np.zeros(n, np.uint8)
    assert np.array_equal(scan_i8(mmv, ones, f), np.arange(1, n + 1))
    f = np.ones(n, np.uint8)
    x = np.random.default_rng(3).uniform(-1, 1, n).astype(np.float16)
    assert np.array_equal(scan_f16(mmv, x, f), x.astype(np.float32))      # identity, exactly
    # flag byte values other than 1 count, and flag[0] is ignored
    f = np.zeros(n, np.uint8)
    f[[5, 4096, 20000]] = [200, 2, 128]
    assert np.array_equal(scan_i8(mmv, ones, f), oracle.seg_scan_i8(ones, f))


def test_scan_int_wraps_mod_2_32(mmv):
    n = 1 << 25
    x = np.full(n, -128, np.int8)
    f = np.zeros(n, np.uint8)
    got = scan_i8(mmv, x, f)
    assert got[-1] == 0 and got[(1 << 24) - 1] == -2 ** 31 and got[1 << 24] == 2 ** 31 - 128
    assert np.array_equal(got, oracle.seg_scan_i8(x, f))


def test_scan_with_offsets(mmv):
    rng = np.random.default_rng(11)
    lens = rng.integers(0, 300, 700)
    off = gen.offsets_from_lengths(lens)
    n = int(off[-1])
    x = rng.integers(-128, 128, n).astype(np.int8)
    f = oracle.flags_from_offsets(off, n)
    assert np.array_equal(scan_i8(mmv, x, off), oracle.seg_scan_i8(x, f))
    xf = rng.uniform(-1, 1, n).astype(np.float16)
    z, a = oracle.seg_scan_f16(xf, f)
    assert_fp(scan_f16(mmv, xf, off), z, a, "offset-encoded scan")


def test_scan_is_deterministic_for_integers(mmv):
    x, f = gen.config3(1 << 22)
    a = scan_i8(mmv, x, f)
    for _ in range(3):
        assert np.array_equal(scan_i8(mmv, x, f), a)


def test_config1_full(mmv):
    x, f = gen.config1()
    z, a = oracle.seg_scan_f16(x, f)
    assert_fp(scan_f16(mmv, x, f), z, a, "config 1")


def test_config3_reduced_and_config5_cases_reduced(mmv):
    x, f = gen.config3(1 << 24)
    assert np.array_equal(scan_i8(mmv, x, f), oracle.seg_scan_i8(x, f))
    n = 1 << 23
    xv = gen.config5_values(n)
    for case, _ in gen.C5_CASES:
        f = gen.config5_flags(n, case)
        z, a = oracle.seg_scan_f16(xv, f)
        assert_fp(scan_f16(mmv, xv, f), z, a, f"config 5 / {case}")


def test_plain_scan_without_a_flag_vector(mmv):
    # seg = None: one segment, the kernel reads no flags at all; same result as all-zero flags
    rng = np.random.default_rng(7)
    for n in (1, 33, TILE - 1, 3 * TILE + 4099):
        xi = rng.integers(-128, 128, n).astype(np.int8)
        zero = np.zeros(n, np.uint8)
        ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN, mmv.I8_TO_I32, mmv.SEG_FLAGS_U8, n)
        got = mmv.seg_scan(dev(xi), None, workspace=ws).cpu().numpy()
        assert mmv.last_async_status(ws) == 0
        assert np.array_equal(got, oracle.seg_scan_i8(xi, zero))
        xf = rng.uniform(-1, 1, n).astype(np.float16)
        ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN, mmv.F16_TO_F32, mmv.SEG_FLAGS_U8, n)
        got = mmv.seg_scan(dev(xf), None, workspace=ws).cpu().numpy()
        z, a = oracle.seg_scan_f16(xf, zero)
        assert_fp(got, z, a, f"plain scan n={n}")
        # (the floating-point plain scan is a kernel variant of its own: exclusive and bfloat16 too)
        got = mmv.seg_scan(dev(xf), None, exclusive=True).cpu().numpy()
        e, ea = oracle.seg_scan_excl_f16(xf, zero)
        assert_fp(got, e, ea, f"plain exclusive scan n={n}")
        xb = gen.bf16_normal(9, n)
        for exclusive in (False, True):
            got = mmv.seg_scan(dev_bf16(xb), None, exclusive=exclusive).cpu().numpy()
            zb, ab = oracle.seg_scan_bf16(xb, zero, exclusive=exclusive)
            assert_fp(got, zb, ab, f"plain bf16 scan n={n} exclusive={exclusive}")
    for n in (7 * TILE + 5, 40 * TILE + 31):                   # many tiles per warpgroup, a ragged end
        xf = rng.uniform(-1, 1, n).astype(np.float16)
        z, a = oracle.seg_scan_f16(xf, np.zeros(n, np.uint8))
        assert_fp(mmv.seg_scan(dev(xf), None).cpu().numpy(), z, a, f"plain scan n={n}")
    # host vectors, chunked, no flags
    n = 9 * TILE + 17
    xf = rng.uniform(-1, 1, n).astype(np.float16)
    scratch = mmv.host_scan_scratch(mmv.F16_TO_F32, 2 * TILE)
    out = mmv.seg_scan_host(torch.from_numpy(xf).pin_memory(), None, chunk=2 * TILE, scratch=scratch)
    assert mmv.last_async_status(scratch) == 0
    z, a = oracle.seg_scan_f16(xf, np.zeros(n, np.uint8))
    assert_fp(out.numpy(), z, a, "plain host scan")


def _mixed_magnitude_segments(rng, nseg, max_len, small=1e-3, large=2e3):
    """Segments of small values right behind segments of large ones (lengths 1..max_len, skewed to short)."""
    lens = np.minimum(max_len, 1 + (rng.pareto(0.6, nseg) * 2).astype(np.int64))
    lens[rng.integers(0, nseg, 8)] = max_len                       # a few of the longest, too
    off = gen.offsets_from_lengths(lens)
    n = int(off[-1])
    scale = np.where(np.arange(nseg) % 2 == 0, large, small)       # every other segment is small
    v = rng.standard_normal(n) * np.repeat(scale, lens)
    f = oracle.flags_from_offsets(off, n)
    return v, f, off


def test_scan_tiny_segments_next_to_large_values(mmv):
    # Floating-point addition is not a group (Section 2): prefix(j) - prefix(last start - 1) leaves a segment of
    # values 1e-3 behind a segment of values 2e3 in the rounding of the prefixes, while the bound is relative to
    # the segment's own sum of magnitudes.  Segment lengths 1 .. 5000: inside a row, across rows, pieces, units
    # and tiles; inclusive and exclusive, flag- and offset-encoded, fp16 and bfloat16, device and host vectors.
    rng = np.random.default_rng(2024)
    v, f, off = _mixed_magnitude_segments(rng, 9000, 5000)
    n = v.shape[0]
    assert n > 20 * TILE
    x = v.astype(np.float16)
    z, a = oracle.seg_scan_f16(x, f)
    assert_fp(scan_f16(mmv, x, f), z, a, "fp16 inclusive")
    assert_fp(scan_f16(mmv, x, off), z, a, "fp16 inclusive, offsets")
    e, ea = oracle.seg_scan_excl_f16(x, f)
    assert_fp(scan_f16(mmv, x, f, exclusive=True), e, ea, "fp16 exclusive")
    xb = gen.bf16_bits_of(v.astype(np.float32))
    for exclusive in (False, True):
        zb, ab = oracle.seg_scan_bf16(xb, f, exclusive=exclusive)
        got = mmv.seg_scan(dev_bf16(xb), dev(f), exclusive=exclusive).cpu().numpy()
        assert_fp(got, zb, ab, f"bf16 exclusive={exclusive}")
    chunk = 4 * TILE
    scratch = mmv.host_scan_scratch(mmv.F16_TO_F32, chunk)
    out = mmv.seg_scan_host(torch.from_numpy(x).pin_memory(), torch.from_numpy(f).pin_memory(), chunk=chunk, scratch=scratch)
    assert mmv.last_async_status(scratch) == 0
    assert_fp(out.numpy(), z, a, "fp16 host vectors")
    # dense starts: most rows of the layout hold several segments of both magnitudes
    v, f, _ = _mixed_magnitude_segments(rng, 120000, 12)
    x = v.astype(np.float16)
    z, a = oracle.seg_scan_f16(x, f)
    assert_fp(scan_f16(mmv, x, f), z, a, "fp16 inclusive, short segments")
    e, ea = oracle.seg_scan_excl_f16(x, f)
    assert_fp(scan_f16(mmv, x, f, exclusive=True), e, ea, "fp16 exclusive, short segments")


def test_scan_mixed_magnitudes_inside_a_segment(mmv):
    # The bound of an element is relative to the magnitudes IN FRONT of it in its segment: small values that
    # open a segment keep a small bound even when large values follow in the same row, piece or unit, and
    # large values that cancel (+a, -a) in front of a start must not leak into the segment behind it.
    rng = np.random.default_rng(77)
    n = 9 * TILE + 1500
    v = rng.standard_normal(n) * 1e-3
    f = (rng.random(n) < 0.004).astype(np.uint8)
    starts = np.flatnonzero(f)
    for s in starts[::3]:                                  # large values from the 3rd .. 40th element of a segment on
        k = s + rng.integers(2, 40)
        m = v[k:k + rng.integers(1, 200)].shape[0]
        v[k:k + m] = rng.standard_normal(m) * 2e3
    for s in starts[1::3]:                                 # a cancelling pair right in front of a start
        if s >= 2:
            v[s - 2], v[s - 1] = 3000.0, -3000.0
    x = v.astype(np.float16)
    z, a = oracle.seg_scan_f16(x, f)
    assert_fp(scan_f16(mmv, x, f), z, a, "inclusive")
    e, ea = oracle.seg_scan_excl_f16(x, f)
    assert_fp(scan_f16(mmv, x, f, exclusive=True), e, ea, "exclusive")
    # no start at all in long stretches: small leading values of the vector, large ones later (plain scan too)
    v = rng.standard_normal(n) * 1e-3
    v[3 * TILE + 517:] *= 1e6
    x = v.astype(np.float16)
    zero = np.zeros(n, np.uint8)
    z, a = oracle.seg_scan_f16(x, zero)
    assert_fp(scan_f16(mmv, x, zero), z, a, "one segment, flag vector")
    assert_fp(mmv.seg_scan(dev(x), None).cpu().numpy(), z, a, "one segment, no flag vector")


# ---------------------------------------------------------------------------
# scan of host-resident vectors, chunk by chunk (carry handed from chunk to chunk on the device)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("n,chunk,p", [(5 * TILE + 123, TILE, 0.0), (5 * TILE + 123, TILE, 1e-3), (7 * TILE, 2 * TILE, 0.3),
                                       (TILE - 5, TILE, 0.01), (40 * TILE + 1, 8 * TILE, 1e-5), (3 * TILE, 4 * TILE, 0.5)])
def test_scan_of_host_vectors_in_chunks(mmv, n, chunk, p):
    rng = np.random.default_rng(n + chunk)
    f = (rng.random(n) < p).astype(np.uint8)
    f[::chunk] |= (rng.random(f[::chunk].shape[0]) < 0.5).astype(np.uint8)      # some chunks start a segment, some continue
    xi = rng.integers(-128, 128, n).astype(np.int8)
    xf = rng.uniform(-1, 1, n).astype(np.float16)
    for x in (xi, xf):
        xh, fh = torch.from_numpy(x).pin_memory(), torch.from_numpy(f).pin_memory()
        scratch = mmv.host_scan_scratch(mmv.I8_TO_I32 if x.dtype == np.int8 else mmv.F16_TO_F32, chunk)
        out = mmv.seg_scan_host(xh, fh, chunk=chunk, scratch=scratch)
        assert mmv.last_async_status(scratch) == 0            # synchronises the stream
        got = out.numpy()
        if x.dtype == np.int8:
            assert np.array_equal(got, oracle.seg_scan_i8(x, f))
        else:
            z, a = oracle.seg_scan_f16(x, f)
            assert_fp(got, z, a, f"host scan n={n} chunk={chunk} p={p}")


# ---------------------------------------------------------------------------
# segmented sum over CSR offsets
# ---------------------------------------------------------------------------
def sum_csr(mmv, x, off, guard=16):
    n, nseg = x.shape[0], off.shape[0] - 1
    dt = mmv.F16_TO_F32 if x.dtype == np.float16 else mmv.I8_TO_I32
    ws = mmv.alloc_workspace(mmv.OP_SEG_SUM, dt, mmv.SEG_OFFSETS_I32, n, nseg)
    tdt = torch.float32 if x.dtype == np.float16 else torch.int32
    buf = torch.full((nseg + guard,), -777, dtype=tdt, device="cuda")
    xd = dev(x) if n else torch.empty(0, dtype=torch.float16 if x.dtype == np.float16 else torch.int8, device="cuda")
    mmv.seg_sum(xd, dev(off), out=buf[:nseg], workspace=ws)
    assert mmv.last_async_status(ws) == 0
    got = buf.cpu().numpy()
    assert (got[nseg:] == -777).all()
    return got[:nseg]


@pytest.mark.parametrize("maxlen,nseg", [(1, 5000), (3, 40000), (40, 3000), (700, 300), (5000, 60), (40000, 9)])
def test_seg_sum_csr_random_lengths(mmv, maxlen, nseg):
    rng = np.random.default_rng(maxlen)
    lens = rng.integers(0, maxlen + 1, nseg)
    off = gen.offsets_from_lengths(lens)
    n = int(off[-1])
    x = rng.integers(-128, 128, n).astype(np.int8)
    assert np.array_equal(sum_csr(mmv, x, off), oracle.seg_sum_csr_i8(x, off))
    xf = rng.standard_normal(n).astype(np.float16)
    want, a = oracle.seg_sum_csr_f16(xf, off)
    got = sum_csr(mmv, xf, off)
    assert_fp(got, want, a, f"maxlen={maxlen}")
    assert (got[lens == 0] == 0).all()


def test_seg_sum_csr_edges(mmv):
    g = __import__("conftest").load_golden("csr_examples.txt")
    x = np.asarray(g["sum_x"], np.int8)
    off = np.asarray(g["sum_off"], np.int32)
    assert sum_csr(mmv, x, off).tolist() == g["sum_out"]
    # one segment covering everything; boundaries exactly on row / piece / span / tile edges
    n = 3 * TILE + 5
    x = np.random.default_rng(1).integers(-128, 128, n).astype(np.int8)
    assert np.array_equal(sum_csr(mmv, x, np.asarray([0, n], np.int32)), oracle.seg_sum_csr_i8(x, np.asarray([0, n], np.int32)))
    off = np.asarray([0, 0, 32, 1024, 1024, 4096, TILE, TILE, TILE + 1, 2 * TILE + 4096, n, n, n], np.int32)
    assert np.array_equal(sum_csr(mmv, x, off), oracle.seg_sum_csr_i8(x, off))
    # segments that do not cover the ends of x: values outside [off[0], off[-1]) are ignored
    off = np.asarray([100, 5000, 5000, 40000], np.int32)
    assert np.array_equal(sum_csr(mmv, x, off), oracle.seg_sum_csr_i8(x, off))
    # segments that span more than 32 spans each, and more than 32 spans of ignored values at both ends
    n = 150 * 4096 + 77
    x = np.random.default_rng(2).integers(-128, 128, n).astype(np.int8)
    off = np.asarray([34 * 4096 + 5, 34 * 4096 + 7, 70 * 4096, 70 * 4096 + 1, 110 * 4096 + 4095, 110 * 4096 + 4095], np.int32)
    assert np.array_equal(sum_csr(mmv, x, off), oracle.seg_sum_csr_i8(x, off))
    off = np.asarray([0, 33 * 4096, n], np.int32)
    assert np.array_equal(sum_csr(mmv, x, off), oracle.seg_sum_csr_i8(x, off))
    # all segments empty, no values at all
    off = np.zeros(9, np.int32)
    assert sum_csr(mmv, np.zeros(0, np.int8), off).tolist() == [0] * 8


def test_seg_sum_tiny_segments_next_to_large_values(mmv):
    # segments of 1..4 small values between large ones: a difference of two prefixes would lose them in
    # rounding (the bound is relative to the segment's own sum of magnitudes), so such sums have to come
    # from the input values themselves; dense boundaries, every row of the tile layout has several
    rng = np.random.default_rng(7)
    nseg = 60000
    lens = rng.integers(1, 9, nseg)
    off = gen.offsets_from_lengths(lens)
    n = int(off[-1])
    big = rng.integers(0, 2, nseg).astype(bool)                      # every other segment holds large values
    scale = np.where(big, 2000.0, 1e-3)
    x = (rng.standard_normal(n) * np.repeat(scale, lens)).astype(np.float16)
    want, a = oracle.seg_sum_csr_f16(x, off)
    got = sum_csr(mmv, x, off)
    assert_fp(got, want, a, "tiny next to large")
    # the same with segment boundaries exactly at row, piece and span edges and lengths up to 32 (a segment
    # inside one or two adjacent 32-element rows: the reach of the kernel's cancellation check)
    lens = rng.integers(1, 33, 20000)
    lens[::7] = 32
    off = gen.offsets_from_lengths(lens)
    n = int(off[-1])
    scale = np.where(rng.integers(0, 3, lens.shape[0]) == 0, 3000.0, 2e-3)
    x = (rng.standard_normal(n) * np.repeat(scale, lens)).astype(np.float16)
    want, a = oracle.seg_sum_csr_f16(x, off)
    assert_fp(sum_csr(mmv, x, off), want, a, "tiny next to large, longer")


@pytest.mark.parametrize("tiny_len", [5, 10, 20, 32])
def test_seg_sum_short_tiny_segments_between_long_large_ones(mmv, tiny_len):
    # spans with few boundaries (long segments of magnitude 2e3) that also hold a segment of 5 to 32 values of
    # magnitude 1e-3: a difference of the span's prefixes would lose it; the stated bound holds for it at any
    # magnitudes
    rng = np.random.default_rng(tiny_len)
    lens = []
    while sum(lens) < 6 * TILE:
        lens += [int(rng.integers(1200, 1800)), tiny_len]
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    n = int(off[-1])
    scale = np.repeat(np.where(np.arange(len(lens)) % 2 == 0, 2e3, 1e-3), lens)
    x = (rng.standard_normal(n) * scale).astype(np.float16)
    want, a = oracle.seg_sum_csr_f16(x, off)
    got = sum_csr(mmv, x, off)
    short = np.diff(off) <= 32
    assert_fp(got[short], want[short], a[short], f"short segments of {tiny_len}")
    # the products of SpMV take the same path (pairs of bf16 values): rows of the same lengths
    col = rng.integers(0, 1000, n).astype(np.int32)
    val = (rng.standard_normal(n) * scale).astype(np.float16)
    xv = rng.standard_normal(1000).astype(np.float32)
    wy, ay = oracle.spmv_csr(off, col, val, xv)
    gy = mmv.spmv_csr(dev(off), dev(col), dev(val), dev(xv)).cpu().numpy()
    assert_fp(gy[short], wy[short], ay[short], f"short rows of {tiny_len}")


@pytest.mark.parametrize("seed", [1, 2])
def test_seg_sum_short_segments_of_any_magnitude_random(mmv, seed):
    # per-segment magnitudes 1e-3, 1 or 2e3 at random; four laws of segment lengths (few boundaries per span,
    # dozens, many, long segments with clusters of short ones); every segment of up to 32 elements holds the bound
    rng = np.random.default_rng(seed)
    for trial in range(24):
        n_target = int(rng.choice([3 * TILE, 7 * TILE + 123]))
        mode = trial % 4
        lens, tot = [], 0
        while tot < n_target:
            if mode == 0:
                l = int(rng.choice([rng.integers(1, 33), rng.integers(300, 3000)], p=[0.3, 0.7]))
            elif mode == 1:
                l = int(rng.choice([rng.integers(1, 33), rng.integers(60, 400)], p=[0.4, 0.6]))
            elif mode == 2:
                l = int(rng.integers(1, 40))
            else:
                l = int(rng.choice([rng.integers(1, 33), rng.integers(3000, 20000)], p=[0.6, 0.4]))
            lens.append(l)
            tot += l
        off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
        scale = np.repeat(rng.choice([1e-3, 1.0, 2e3], len(lens), p=[0.3, 0.3, 0.4]), lens)
        x = (rng.standard_normal(int(off[-1])) * scale).astype(np.float16)
        want, a = oracle.seg_sum_csr_f16(x, off)
        mmv.debug_force_sum_groups(int(rng.choice([0, 2, 3])))
        try:
            got = sum_csr(mmv, x, off)
        finally:
            mmv.debug_force_sum_groups(0)
        short = np.asarray(lens) <= 32
        assert_fp(got[short], want[short], a[short], f"trial {trial}, law {mode}")


def test_seg_sum_long_segments_at_the_edge_of_the_stated_magnitude_range(mmv):
    # What the header promises for segments LONGER than two 32-element rows: the bound holds when the magnitudes
    # inside a 4096-element span are within about 2^10 of each other.  Segments of 40 .. 3000 elements, every
    # other one scaled by 2^-10 (so that a small segment's partial rows are differences of prefixes that still
    # carry its big neighbour's values), also through SpMV's bf16-pair path.
    rng = np.random.default_rng(41)
    lens = rng.integers(40, 3000, 4000)
    lens[::5] = rng.integers(33, 70, lens[::5].shape[0])         # many just beyond the reach of the cancellation check
    off = gen.offsets_from_lengths(lens)
    n = int(off[-1])
    scale = np.where(np.arange(lens.shape[0]) % 2 == 0, 1.0, 2.0 ** -10)
    x = (rng.standard_normal(n) * np.repeat(scale, lens)).astype(np.float16)
    want, a = oracle.seg_sum_csr_f16(x, off)
    assert_fp(sum_csr(mmv, x, off), want, a, "long segments, magnitudes 2^10 apart")
    val = x
    cols = n
    col = np.arange(n, dtype=np.int32)
    xv = np.ones(cols, np.float32)
    wanty, ay = oracle.spmv_csr(off, col, val, xv)
    assert_fp(spmv(mmv, off, col, val, xv), wanty, ay, "SpMV rows, magnitudes 2^10 apart")


def test_seg_sum_long_runs_of_empty_segments(mmv):
    # hundreds of thousands of empty segments in a row (at the start, in the middle of a span, exactly on a
    # span edge, at the end): the kernel jumps over such runs instead of visiting them one by one
    rng = np.random.default_rng(99)
    n = 6 * TILE + 1000
    cuts = np.sort(rng.choice(np.arange(1, n), 40, replace=False))
    pieces = [np.zeros(300000, np.int64)]                                   # leading run at 0
    for c in cuts:
        pieces.append(np.asarray([c], np.int64))
    pieces.append(np.full(250000, 2 * TILE + 777, np.int64))                # inside a span
    pieces.append(np.full(250000, 3 * TILE, np.int64))                      # on a tile edge
    pieces.append(np.full(400000, n, np.int64))                             # trailing run at n
    off = np.sort(np.concatenate(pieces + [np.asarray([0, n], np.int64)])).astype(np.int32)
    x = rng.integers(-128, 128, n).astype(np.int8)
    want = oracle.seg_sum_csr_i8(x, off)
    import time
    t0 = time.time()
    got = sum_csr(mmv, x, off)
    assert np.array_equal(got, want)
    xf = rng.standard_normal(n).astype(np.float16)
    wantf, a = oracle.seg_sum_csr_f16(xf, off)
    assert_fp(sum_csr(mmv, xf, off), wantf, a, "runs of empty segments")
    assert time.time() - t0 < 5.0


@pytest.mark.parametrize("seed", [1, 2, 3, 4])
def test_seg_sum_mixed_runs_and_lengths_stress(mmv, seed):
    # random mixtures of segment lengths (tiny, medium, long) and of runs of empty segments whose lengths sit
    # around the batch and table sizes of the kernel (31..33, 63..65, 127..130, a few thousand), some of
    # them pinned to row, piece, span and tile edges
    rng = np.random.default_rng(seed)
    n = 5 * TILE + int(rng.integers(0, 5000))
    cuts = set(int(c) for c in rng.choice(np.arange(1, n), 300, replace=False))
    cuts |= {32, 1024, 4096, TILE, 2 * TILE + 4096, 3 * TILE - 32, 4 * TILE + 1024, n - 1}
    # a stretch of tiny segments
    a = int(rng.integers(TILE, 2 * TILE))
    cuts |= set(range(a, a + 700, int(rng.integers(1, 4))))
    pos = np.asarray(sorted(c for c in cuts if 0 < c < n), np.int64)
    reps = np.ones(pos.shape[0], np.int64)
    run_lengths = [31, 32, 33, 63, 64, 65, 127, 128, 129, 130, 257, 3000, 5000]
    where = rng.choice(pos.shape[0], len(run_lengths), replace=False)
    for w, r in zip(where, run_lengths):
        reps[w] = r
    edge_idx = [int(np.searchsorted(pos, e)) for e in (4096, TILE, 3 * TILE - 32)]
    for i, r in zip(edge_idx, (40, 129, 1000)):
        reps[i] = r
    body = np.repeat(pos, reps)
    lead = int(rng.integers(0, 200))
    trail = int(rng.integers(0, 200))
    off = np.concatenate([np.zeros(1 + lead, np.int64), body, np.full(1 + trail, n, np.int64)]).astype(np.int32)
    x = rng.integers(-128, 128, n).astype(np.int8)
    assert np.array_equal(sum_csr(mmv, x, off), oracle.seg_sum_csr_i8(x, off))
    xf = rng.standard_normal(n).astype(np.float16)
    want, a_ = oracle.seg_sum_csr_f16(xf, off)
    assert_fp(sum_csr(mmv, xf, off), want, a_, f"stress seed {seed}")
    for groups in (2, 3):
        mmv.debug_force_sum_groups(groups)
        try:
            assert np.array_equal(sum_csr(mmv, x, off), oracle.seg_sum_csr_i8(x, off))
        finally:
            mmv.debug_force_sum_groups(0)


@pytest.mark.parametrize("maxlen", [3, 60, 3000])
def test_seg_sum_csr_many_tiles_per_cta(mmv, maxlen):
    # more tiles than 2 x 148, so every CTA runs several tiles back to back in both warpgroups
    rng = np.random.default_rng(1000 + maxlen)
    n = (1 << 23) + 4321
    lens = rng.integers(0, maxlen + 1, int(2.2 * n / maxlen) + 10)
    cs = np.cumsum(lens)
    keep = int(np.searchsorted(cs, n, side="right"))
    off = np.concatenate([[0], cs[:keep], [n]]).astype(np.int32)
    x = rng.integers(-128, 128, n).astype(np.int8)
    assert np.array_equal(sum_csr(mmv, x, off), oracle.seg_sum_csr_i8(x, off))
    xf = rng.standard_normal(n).astype(np.float16)
    want, a = oracle.seg_sum_csr_f16(xf, off)
    assert_fp(sum_csr(mmv, xf, off), want, a, f"many tiles, maxlen={maxlen}")


@pytest.mark.parametrize("groups", [2, 3])
def test_seg_sum_both_kernel_shapes(mmv, groups):
    # the kernel exists with 8 and with 12 epilogue warps; the library picks by average segment
    # length, here each shape is forced over sparse, dense and empty-heavy boundaries
    mmv.debug_force_sum_groups(groups)
    try:
        for maxlen, nseg in [(2, 200000), (90, 40000), (6000, 1500), (70000, 40)]:
            rng = np.random.default_rng(groups * 100 + maxlen)
            lens = rng.integers(0, maxlen + 1, nseg)
            off = gen.offsets_from_lengths(lens)
            n = int(off[-1])
            x = rng.integers(-128, 128, n).astype(np.int8)
            assert np.array_equal(sum_csr(mmv, x, off), oracle.seg_sum_csr_i8(x, off))
            xf = rng.standard_normal(n).astype(np.float16)
            want, a = oracle.seg_sum_csr_f16(xf, off)
            assert_fp(sum_csr(mmv, xf, off), want, a, f"groups={groups} maxlen={maxlen}")
    finally:
        mmv.debug_force_sum_groups(0)


def test_seg_sum_config2_reduced(mmv):
    x, off = gen.config2(1 << 22)
    want, a = oracle.seg_sum_csr_f16(x, off)
    assert_fp(sum_csr(mmv, x, off), want, a, "config 2 (n = 2^22)")


# ---------------------------------------------------------------------------
# segmented sum over start flags (COMPRESS of the flags, then the offset kernel)
# ---------------------------------------------------------------------------
def sum_flags(mmv, x, f, guard=16):
    n = x.shape[0]
    dt = mmv.F16_TO_F32 if x.dtype == np.float16 else mmv.I8_TO_I32
    ws = mmv.alloc_workspace(mmv.OP_SEG_SUM, dt, mmv.SEG_FLAGS_U8, n)
    tdt = torch.float32 if x.dtype == np.float16 else torch.int32
    buf = torch.full((n + guard,), -777, dtype=tdt, device="cuda")
    k = torch.full((1,), -1, dtype=torch.int64, device="cuda")
    mmv.seg_sum(dev(x), dev(f), out=buf[:n], num_segments=k, workspace=ws)
    assert mmv.last_async_status(ws) == 0
    got, kk = buf.cpu().numpy(), int(k.item())
    assert (got[kk:] == -777).all()          # nothing beyond the K sums is written
    return got[:kk]


@pytest.mark.parametrize("n,p", [(1, 0.5), (31, 0.3), (4097, 0.01), (3 * TILE + 777, 0.0), (3 * TILE + 777, 1e-3),
                                 (5 * TILE + 13, 0.2), (2 * TILE, 1.0), ((1 << 22) + 5, 1e-4), ((1 << 21) + 99, 0.6)])
def test_seg_sum_flags(mmv, n, p):
    rng = np.random.default_rng(int(n * 7 + p * 1000))
    f = (rng.random(n) < p).astype(np.uint8) * rng.integers(1, 256, n).astype(np.uint8)   # any non-zero byte counts
    x = rng.integers(-128, 128, n).astype(np.int8)
    want = oracle.seg_sum_flags_i8(x, f)
    got = sum_flags(mmv, x, f)
    assert got.shape == want.shape and np.array_equal(got, want)
    xf = rng.standard_normal(n).astype(np.float16)
    wantf, a = oracle.seg_sum_flags_f16(xf, f)
    gotf = sum_flags(mmv, xf, f)
    assert gotf.shape == wantf.shape
    assert_fp(gotf, wantf, a, f"flag-form seg-sum n={n} p={p}")


def test_seg_sum_flags_matches_paper_example(mmv):
    g = __import__("conftest").load_golden("sec2_worked_example.txt")
    x = np.asarray(g["x"], np.int8)
    f = np.asarray(g["f"], np.uint8)
    assert sum_flags(mmv, x, f).tolist() == g["seg_sum"]


# ---------------------------------------------------------------------------
# CSR SpMV
# ---------------------------------------------------------------------------
def spmv(mmv, rowptr, col, val, x):
    rows = rowptr.shape[0] - 1
    ws = mmv.alloc_workspace(mmv.OP_SPMV_CSR, mmv.F16_TO_F32, mmv.SEG_OFFSETS_I32, val.shape[0], rows)
    y = mmv.spmv_csr(dev(rowptr), dev(col), dev(val), dev(x), workspace=ws)
    assert mmv.last_async_status(ws) == 0
    return y.cpu().numpy()


def test_spmv_golden_and_random(mmv):
    g = __import__("conftest").load_golden("csr_examples.txt")
    y = spmv(mmv, np.asarray(g["spmv_rowptr"], np.int32), np.asarray(g["spmv_col"], np.int32),
             np.asarray(g["spmv_val"], np.float32).astype(np.float16), np.asarray(g["spmv_x"], np.float32))
    assert y.tolist() == g["spmv_y"]
    for rows, frac in ((3000, 0.0), (20000, 0.1), (1 << 17, 0.05)):
        rowptr, col, val, x = gen.config4(rows=rows, empty_fraction=frac)
        want, a = oracle.spmv_csr(rowptr, col, val, x)
        got = spmv(mmv, rowptr, col, val, x)
        assert_fp(got, want, a, f"spmv rows={rows}")
        assert (got[np.diff(rowptr) == 0] == 0).all()


@pytest.mark.parametrize("block", gen.BSA_BLOCKS)
@pytest.mark.parametrize("random_blocks", gen.BSA_RANDOM)
def test_spmv_block_sparse_attention(mmv, block, random_blocks):
    # the blocked sparse-attention matrices of Section 5 (global, window and random blocks), reduced to 8192 rows
    rowptr, col, val, x = gen.block_sparse_attention_csr(block, random_blocks, dim=8192)
    want, a = oracle.spmv_csr(rowptr, col, val, x)
    assert_fp(spmv(mmv, rowptr, col, val, x), want, a, f"b-{block}_r-{random_blocks}")


@pytest.mark.parametrize("kind", gen.ROW_LENGTH_MIXES)
def test_seg_sum_row_length_mixes(mmv, kind):
    # segment lengths with the minimum / average / maximum of the matrices of Table 5.1
    x, off = gen.seg_sum_row_mix(kind, 3 << 20)
    want, a = oracle.seg_sum_csr_f16(x, off)
    assert_fp(sum_csr(mmv, x, off), want, a, kind)
    xi = gen.i8_uniform(7, x.shape[0])
    assert np.array_equal(sum_csr(mmv, xi, off), oracle.seg_sum_csr_i8(xi, off))


# ---------------------------------------------------------------------------
# COMPRESS (Section 2)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("n", [1, 63, 64, 65, TILE - 1, TILE, TILE + 1, 5 * TILE + 333])
@pytest.mark.parametrize("p", [0.0, 0.01, 0.5, 1.0])
def test_compress(mmv, n, p):
    rng = np.random.default_rng(n + int(100 * p))
    f = ((rng.random(n) < p) * rng.integers(1, 256, n)).astype(np.uint8)        # any non-zero byte keeps the element
    for x in (rng.integers(-128, 128, n).astype(np.int8), rng.standard_normal(n).astype(np.float16)):
        want = oracle.compress(x, f)
        guard = torch.full((n + 8,), 77, dtype=torch.from_numpy(x[:1]).dtype, device="cuda")
        out, count = mmv.compress(dev(x), dev(f), out=guard[:n])
        k = int(count.item())
        got = guard.cpu().numpy()
        assert k == want.shape[0]
        assert np.array_equal(got[:k].view(np.uint8), want.view(np.uint8))          # bit for bit
        assert (got[max(k, 0):] == 77).all() if k == n else (got[n:] == 77).all()   # nothing past the end
    xb = gen.bf16_normal(3, n)
    out, count = mmv.compress(dev_bf16(xb), dev(f))
    k = int(count.item())
    assert np.array_equal(out[:k].view(torch.int16).cpu().numpy().view(np.uint16), oracle.compress(xb, f))


def test_compress_with_dense_and_sparse_stretches(mmv):
    # stretches of 2048 elements (one warp's share of a chunk) with 0, a few, 127, 128, 129, half and all flags
    # set, in random order: both routes of the scatter pass, every phase of the output inside a 16-byte vector
    rng = np.random.default_rng(5)
    counts = [0, 1, 3, 40, 127, 128, 129, 500, 1024, 2047, 2048]
    for trial in range(3):
        pieces = []
        for _ in range(40):
            k = int(rng.choice(counts))
            piece = np.zeros(2048, np.uint8)
            piece[rng.choice(2048, k, replace=False)] = rng.integers(1, 256, k)
            pieces.append(piece)
        f = np.concatenate(pieces)[: 40 * 2048 - int(rng.integers(0, 2048))]
        n = f.shape[0]
        for x in (rng.integers(-128, 128, n).astype(np.int8), rng.standard_normal(n).astype(np.float16)):
            want = oracle.compress(x, f)
            guard = torch.full((n + 8,), 77, dtype=torch.from_numpy(x[:1]).dtype, device="cuda")
            out, count = mmv.compress(dev(x), dev(f), out=guard[:n])
            k = int(count.item())
            got = guard.cpu().numpy()
            assert k == want.shape[0]
            assert np.array_equal(got[:k].view(np.uint8), want.view(np.uint8))
            assert (got[n:] == 77).all()
        # the same flags as segment starts of a flag-encoded segmented sum (positions instead of values)
        xi = gen.i8_uniform(9, n)
        kd = torch.zeros(1, dtype=torch.int64, device="cuda")
        got = mmv.seg_sum(dev(xi), dev(f), num_segments=kd)
        want = oracle.seg_sum_flags_i8(xi, f)
        assert int(kd.item()) == want.shape[0]
        assert np.array_equal(got[: want.shape[0]].cpu().numpy(), want)


def test_calls_with_nothing_to_do_leave_ok_in_a_fresh_workspace(mmv):
    # a workspace that no call has used yet (all bytes set) is handed to calls without elements, segments, rows
    # or non-zeros: the status read back afterwards is MMV_OK, not whatever the memory held
    def fresh():
        return torch.full((4096,), 0xFF, dtype=torch.uint8, device="cuda")
    e16 = torch.empty(0, dtype=torch.float16, device="cuda")
    e8 = torch.empty(0, dtype=torch.uint8, device="cuda")
    ws = fresh()
    mmv.seg_scan(e16, e8, workspace=ws)
    assert mmv.last_async_status(ws) == 0
    ws = fresh()
    mmv.seg_scan_minmax(e16, e8, workspace=ws)
    assert mmv.last_async_status(ws) == 0
    ws = fresh()
    mmv.compress(e16, e8, workspace=ws)
    assert mmv.last_async_status(ws) == 0
    ws = fresh()
    out = mmv.seg_sum(e16, torch.zeros(4, dtype=torch.int32, device="cuda"), workspace=ws)      # three empty segments
    assert out.cpu().tolist() == [0.0, 0.0, 0.0] and mmv.last_async_status(ws) == 0
    ws = fresh()
    y = mmv.spmv_csr(torch.zeros(3, dtype=torch.int32, device="cuda"), torch.empty(0, dtype=torch.int32, device="cuda"), e16,
                     torch.ones(5, dtype=torch.float32, device="cuda"), workspace=ws)                # two rows, no non-zeros
    assert y.cpu().tolist() == [0.0, 0.0] and mmv.last_async_status(ws) == 0


def test_compress_of_the_paper_example(mmv):
    g = __import__("conftest").load_golden("sec2_worked_example.txt")
    out, count = mmv.compress(dev(np.asarray(g["x"], np.int8)), dev(np.asarray(g["f"], np.uint8)))
    assert out[:int(count.item())].cpu().tolist() == g["compress_x_f"]


# ---------------------------------------------------------------------------
# randomised shapes
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("seed", [11, 12, 13])
def test_seg_sum_random_shapes(mmv, seed):
    # random sizes, segment-length laws (tiny, geometric, wide, with empty segments, with runs of them, constant),
    # leading ignored elements, all three value types and both kernel shapes
    rng = np.random.default_rng(seed)
    for trial in range(40):
        n = int(rng.choice([rng.integers(1, 300), rng.integers(300, 40000), rng.integers(40000, 6 * TILE)]))
        kind = int(rng.integers(0, 6))
        if kind == 0:
            lens = rng.integers(0, 4, 4 * n)
        elif kind == 1:
            lens = rng.geometric(1 / rng.choice([2.0, 6.0, 40.0, 300.0]), 2 * n) - rng.integers(0, 2)
        elif kind == 2:
            lens = rng.integers(1, rng.choice([8, 64, 2000, 20000]), n)
        elif kind == 3:
            lens = rng.integers(1, 50, n)
            lens[rng.random(n) < 0.3] = 0
        elif kind == 4:
            lens = rng.integers(1, 10, n)
            for _ in range(3):
                at = int(rng.integers(0, lens.shape[0]))
                lens = np.concatenate([lens[:at], np.zeros(int(rng.choice([31, 32, 33, 127, 129, 300, 5000])), np.int64), lens[at:]])
        else:
            lens = np.full(n, rng.choice([1, 2, 31, 32, 33, 1024, 4096]))
        lead = int(rng.integers(0, 40)) if rng.random() < 0.3 else 0
        off = np.concatenate([[lead], lead + np.cumsum(np.maximum(lens, 0))])
        off = off[off <= n]
        if off.shape[0] < 2:
            off = np.asarray([0, n])
        off = off.astype(np.int32)
        mmv.debug_force_sum_groups(int(rng.choice([0, 2, 3])))
        try:
            what = f"seed {seed} trial {trial} n={n} kind={kind}"
            which = int(rng.integers(0, 3))
            if which == 0:
                x = rng.integers(-128, 128, n).astype(np.int8)
                assert np.array_equal(sum_csr(mmv, x, off), oracle.seg_sum_csr_i8(x, off)), what
            elif which == 1:
                x = (rng.standard_normal(n) * rng.choice([1.0, 30.0])).astype(np.float16)
                want, a = oracle.seg_sum_csr_f16(x, off)
                assert_fp(sum_csr(mmv, x, off), want, a, what)
            else:
                xb = gen.bf16_bits_of(rng.standard_normal(n).astype(np.float32))
                ws = mmv.alloc_workspace(mmv.OP_SEG_SUM, mmv.BF16_TO_F32, mmv.SEG_OFFSETS_I32, n, off.shape[0] - 1)
                got = mmv.seg_sum(dev_bf16(xb), dev(off), workspace=ws).cpu().numpy()
                assert mmv.last_async_status(ws) == 0
                want, a = oracle.seg_sum_csr_bf16(xb, off)
                assert_fp(got, want, a, what)
        finally:
            mmv.debug_force_sum_groups(0)


def test_spmv_random_shapes(mmv):
    rng = np.random.default_rng(21)
    for trial in range(40):
        rows = int(rng.choice([rng.integers(1, 50), rng.integers(50, 5000), rng.integers(5000, 100000)]))
        cols = int(rng.integers(1, 100000))
        kind = int(rng.integers(0, 4))
        if kind == 0:
            lens = rng.integers(0, 4, rows)
        elif kind == 1:
            lens = rng.geometric(1 / rng.choice([2.0, 6.0, 60.0]), rows) - rng.integers(0, 2)
        elif kind == 2:
            lens = rng.integers(0, rng.choice([8, 200, 5000]), rows)
        else:
            lens = np.full(rows, rng.choice([1, 2, 32, 33]))
        lens = np.maximum(lens, 0)
        if lens.sum() > 2_000_000:
            lens = lens // 8
        rowptr = gen.offsets_from_lengths(lens)
        nnz = int(rowptr[-1])
        col = rng.integers(0, cols, nnz).astype(np.int32)
        val = (rng.standard_normal(nnz) * rng.choice([1.0, 100.0])).astype(np.float16)
        x = (rng.standard_normal(cols) * rng.choice([1.0, 1e-3, 50.0])).astype(np.float32)
        want, a = oracle.spmv_csr(rowptr, col, val, x)
        assert_fp(spmv(mmv, rowptr, col, val, x), want, a, f"trial {trial} rows={rows} nnz={nnz} kind={kind}")


# ---------------------------------------------------------------------------
# segmented running maximum / minimum (exact: every comparison below is for equality)
# ---------------------------------------------------------------------------
MM_TILE = 8192           # elements per status word of that kernel; a CTA pass covers half of it


def minmax(mmv, x, f, want_min, guard=64):
    """The call with a guard band behind the output: nothing past n may be written."""
    import torch
    n = x.shape[0]
    i8 = x.dtype == np.int8
    buf = torch.full((n + guard,), -77, dtype=torch.int32 if i8 else torch.float32, device="cuda")
    mmv.seg_scan_minmax(dev(x), None if f is None else dev(f), want_min=want_min, out=buf[:n])
    torch.cuda.synchronize()
    assert (buf[n:] == -77).all(), "wrote past the end of the output"
    return buf[:n].cpu().numpy()


@pytest.mark.parametrize("n", [1, 15, 16, 17, 511, 513, 4095, 4096, 4097, MM_TILE - 1, MM_TILE, MM_TILE + 1, 16383, 16385,
                               3 * MM_TILE + 5, 40 * MM_TILE + 4100, 600 * MM_TILE + 77])
@pytest.mark.parametrize("p", [0.0, 1e-4, 1e-2, 0.5, 1.0])
def test_seg_scan_minmax(mmv, n, p):
    rng = np.random.default_rng(n * 11 + int(p * 10000))
    f = (rng.random(n) < p).astype(np.uint8)
    xi = rng.integers(-128, 128, n).astype(np.int8)
    xf = rng.standard_normal(n).astype(np.float16)
    for want_min in (False, True):
        assert np.array_equal(minmax(mmv, xi, f, want_min), oracle.seg_scan_minmax_i8(xi, f, want_min))
        assert np.array_equal(minmax(mmv, xf, f, want_min).astype(np.float64), oracle.seg_scan_minmax_f16(xf, f, want_min))


@pytest.mark.parametrize("n", [1, 17, 4097, MM_TILE + 5, 50 * MM_TILE + 123])
@pytest.mark.parametrize("p", [0.0, 1e-3, 0.1, 1.0])
def test_seg_scan_minmax_bf16(mmv, n, p):
    # bfloat16 values over the whole exponent range (far beyond fp16's), exact comparison
    rng = np.random.default_rng(n * 17 + int(p * 1000))
    f = (rng.random(n) < p).astype(np.uint8)
    xb = gen.bf16_bits_of((rng.standard_normal(n) * 10.0 ** rng.integers(-30, 30, n)).astype(np.float32))
    for want_min in (False, True):
        got = mmv.seg_scan_minmax(dev_bf16(xb), dev(f), want_min=want_min).cpu().numpy()
        assert np.array_equal(got.astype(np.float64), oracle.seg_scan_minmax_bf16(xb, f, want_min))
    got = mmv.seg_scan_minmax(dev_bf16(xb), None).cpu().numpy()
    assert np.array_equal(got.astype(np.float64), oracle.seg_scan_minmax_bf16(xb, np.zeros(n, np.uint8)))


def test_seg_scan_minmax_edges_and_long_carries(mmv):
    # a ramp that falls: the running maximum is carried from element 0 across every tile, the minimum is the input
    n = 400 * MM_TILE + 9
    xf = np.linspace(60000.0, -60000.0, n).astype(np.float16)
    got = minmax(mmv, xf, None, False)
    assert (got == np.float32(xf[0])).all()
    assert np.array_equal(minmax(mmv, xf, None, True), xf.astype(np.float32))
    # flags on the edges of threads' 16-element runs, warps (512), CTA passes (4096) and runs; extreme values next to them
    rng = np.random.default_rng(5)
    n = 9 * MM_TILE + 100
    f = np.zeros(n, np.uint8)
    f[[0, 15, 16, 17, 511, 512, 513, 4095, 4096, 4097, MM_TILE - 1, MM_TILE, MM_TILE + 1, 3 * MM_TILE + 15, 5 * MM_TILE, n - 1]] = 1
    xi = rng.integers(-128, 128, n).astype(np.int8)
    xi[[14, 510, MM_TILE - 2, 5 * MM_TILE - 1]] = 127
    xi[[18, 514, MM_TILE + 2, 5 * MM_TILE + 1]] = -128
    xf = rng.standard_normal(n).astype(np.float16)
    xf[[14, MM_TILE - 2]] = np.float16(65504.0)
    xf[[18, MM_TILE + 2]] = np.float16(-65504.0)
    for want_min in (False, True):
        assert np.array_equal(minmax(mmv, xi, f, want_min), oracle.seg_scan_minmax_i8(xi, f, want_min))
        assert np.array_equal(minmax(mmv, xf, f, want_min).astype(np.float64), oracle.seg_scan_minmax_f16(xf, f, want_min))
    # any non-zero byte is a start
    f = np.where(rng.random(n) < 0.02, rng.choice(np.asarray([1, 2, 0x40, 0x7f, 0x80, 0x81, 0xff], np.uint8), n), 0).astype(np.uint8)
    assert np.array_equal(minmax(mmv, xi, f, False), oracle.seg_scan_minmax_i8(xi, f, False))
    assert np.array_equal(minmax(mmv, xf, f, True).astype(np.float64), oracle.seg_scan_minmax_f16(xf, f, True))
    # the worked example of Section 2 (its values, its flags)
    x = np.asarray([2, 2, 3, 3, 1, 3, 1, 2], np.int8)
    fl = np.asarray([1, 0, 1, 0, 0, 1, 0, 0], np.uint8)
    assert minmax(mmv, x, fl, False).tolist() == [2, 2, 3, 3, 3, 3, 3, 3]
    assert minmax(mmv, x, fl, True).tolist() == [2, 2, 3, 3, 1, 3, 1, 1]


# ---------------------------------------------------------------------------
# int8 values with int64 results (no wrap): exact
# ---------------------------------------------------------------------------
WD_TILE = 2048


def scan_wide(mmv, x, f, guard=64):
    import torch
    n = x.shape[0]
    buf = torch.full((n + guard,), -77, dtype=torch.int64, device="cuda")
    mmv.seg_scan_wide(dev(x), None if f is None else dev(f), out=buf[:n])
    torch.cuda.synchronize()
    assert (buf[n:] == -77).all(), "wrote past the end of the output"
    return buf[:n].cpu().numpy()


@pytest.mark.parametrize("n", [1, 15, 16, 17, 511, 513, WD_TILE - 1, WD_TILE, WD_TILE + 1, 4095, 4097, 3 * WD_TILE + 5,
                               40 * WD_TILE + 1234, 1400 * WD_TILE + 77])
@pytest.mark.parametrize("p", [0.0, 1e-4, 1e-2, 0.5, 1.0])
def test_seg_scan_wide(mmv, n, p):
    rng = np.random.default_rng(n * 13 + int(p * 10000))
    f = (rng.random(n) < p).astype(np.uint8)
    xi = rng.integers(-128, 128, n).astype(np.int8)
    assert np.array_equal(scan_wide(mmv, xi, f), oracle.seg_scan_i8_wide(xi, f))


def test_seg_scan_wide_past_the_int32_range_and_edges(mmv):
    # 2^25 + 5 values of -128: the sums pass -2^32 (the int32 scan is back at 0 there); closed form -128 (i + 1)
    n = (1 << 25) + 5
    x = np.full(n, -128, np.int8)
    got = scan_wide(mmv, x, None)
    assert got[-1] == -128 * n and np.array_equal(got, -128 * np.arange(1, n + 1, dtype=np.int64))
    # the same with one start late in the vector and one flag byte that is not 1
    f = np.zeros(n, np.uint8)
    f[(1 << 24) + 3] = 0x80
    assert np.array_equal(scan_wide(mmv, x, f), oracle.seg_scan_i8_wide(x, f))
    # flags on the edges of threads' 16-element runs, warps (512) and tiles; extreme values next to them
    rng = np.random.default_rng(6)
    n = 9 * WD_TILE + 100
    f = np.zeros(n, np.uint8)
    f[[0, 15, 16, 17, 511, 512, 513, WD_TILE - 1, WD_TILE, WD_TILE + 1, 3 * WD_TILE + 15, 5 * WD_TILE, n - 1]] = 1
    xi = rng.integers(-128, 128, n).astype(np.int8)
    assert np.array_equal(scan_wide(mmv, xi, f), oracle.seg_scan_i8_wide(xi, f))
    # its low 32 bits are what the tensor-core scan returns
    assert np.array_equal(scan_wide(mmv, xi, f).astype(np.int32), scan_i8(mmv, xi, f))
    # the worked example of Section 2
    x = np.asarray([2, 2, 3, 3, 1, 3, 1, 2], np.int8)
    fl = np.asarray([1, 0, 1, 0, 0, 1, 0, 0], np.uint8)
    assert scan_wide(mmv, x, fl).tolist() == [2, 4, 3, 6, 7, 3, 4, 6]


def test_wide_lookback_wait_gives_up_with_a_status(mmv):
    n = 40 * TILE
    x = dev(np.ones(n, np.int8))
    ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN_WIDE, mmv.I8_TO_I32, mmv.SEG_FLAGS_U8, n)
    try:
        mmv.debug_configure(20_000_000, 17)           # 20 ms budget, tile 17 stays silent
        mmv.seg_scan_wide(x, None, workspace=ws)
        assert mmv.last_async_status(ws) == 5
    finally:
        mmv.debug_configure(0, -1)
    out = mmv.seg_scan_wide(x, None, workspace=ws)     # and the next call works
    assert mmv.last_async_status(ws) == 0
    assert np.array_equal(out.cpu().numpy(), np.arange(1, n + 1))


# ---------------------------------------------------------------------------
# exclusive variant of the scan
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("n", [1, 31, 32, 33, 1023, 1025, 4096, TILE - 1, TILE, TILE + 1, 3 * TILE + 4097, 11 * TILE + 777])
@pytest.mark.parametrize("p", [0.0, 1e-3, 0.05, 0.5, 1.0])
def test_exclusive_scan(mmv, n, p):
    rng = np.random.default_rng(n * 7 + int(p * 1000))
    f = (rng.random(n) < p).astype(np.uint8)
    xi = rng.integers(-128, 128, n).astype(np.int8)
    assert np.array_equal(scan_i8(mmv, xi, f, exclusive=True), oracle.seg_scan_excl_i8(xi, f))
    xf = rng.standard_normal(n).astype(np.float16)
    want, a = oracle.seg_scan_excl_f16(xf, f)
    got = scan_f16(mmv, xf, f, exclusive=True)
    assert_fp(got, want, a, f"exclusive scan n={n} p={p}")
    assert got[0] == 0.0 and (got[f != 0] == 0.0).all()        # exactly zero at every segment start


def test_exclusive_scan_flags_on_edges_offsets_and_plain(mmv):
    n = 5 * TILE + 100
    rng = np.random.default_rng(3)
    f = np.zeros(n, np.uint8)
    f[[31, 32, 33, 1023, 1024, 4095, 4096, 4097, TILE - 1, TILE, TILE + 1, 2 * TILE + 4096, 4 * TILE, n - 1]] = 1
    xi = rng.integers(-128, 128, n).astype(np.int8)
    assert np.array_equal(scan_i8(mmv, xi, f, exclusive=True), oracle.seg_scan_excl_i8(xi, f))
    xf = gen.f16_uniform(1, n)
    want, a = oracle.seg_scan_excl_f16(xf, f)
    assert_fp(scan_f16(mmv, xf, f, exclusive=True), want, a, "exclusive, flags on edges")
    # the same segments as offsets (with empty segments in between)
    off = np.asarray([0, 0, 31, 32, 33, 33, 1023, 1024, 4095, 4096, 4097, TILE - 1, TILE, TILE + 1, 2 * TILE + 4096,
                      4 * TILE, n - 1, n, n], np.int32)
    assert np.array_equal(scan_i8(mmv, xi, off, exclusive=True), oracle.seg_scan_excl_i8(xi, f))
    # no flag vector: the plain exclusive scan
    ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN, mmv.I8_TO_I32, mmv.SEG_FLAGS_U8, n)
    got = mmv.seg_scan(dev(xi), None, workspace=ws, exclusive=True).cpu().numpy()
    assert np.array_equal(got, oracle.seg_scan_excl_i8(xi, np.zeros(n, np.uint8)))


# ---------------------------------------------------------------------------
# bfloat16 input values
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("n", [1, 33, 4097, TILE + 5, 7 * TILE + 1234])
@pytest.mark.parametrize("p", [0.0, 1e-3, 0.1, 1.0])
def test_bf16_scan_and_sum(mmv, n, p):
    rng = np.random.default_rng(n + int(p * 1e4))
    f = (rng.random(n) < p).astype(np.uint8)
    xb = gen.bf16_normal(8, n)
    xd, fd = dev_bf16(xb), dev(f)
    for exclusive in (False, True):
        ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN, mmv.BF16_TO_F32, mmv.SEG_FLAGS_U8, n)
        got = mmv.seg_scan(xd, fd, workspace=ws, exclusive=exclusive).cpu().numpy()
        assert mmv.last_async_status(ws) == 0
        want, a = oracle.seg_scan_bf16(xb, f, exclusive=exclusive)
        assert_fp(got, want, a, f"bf16 scan n={n} p={p} exclusive={exclusive}")
    # the same segments as offsets and as flags through the segmented sum
    starts = np.flatnonzero(f)
    off = np.unique(np.concatenate([[0], starts, [n]])).astype(np.int32)
    want, a = oracle.seg_sum_csr_bf16(xb, off)
    ws = mmv.alloc_workspace(mmv.OP_SEG_SUM, mmv.BF16_TO_F32, mmv.SEG_OFFSETS_I32, n, off.shape[0] - 1)
    got = mmv.seg_sum(xd, dev(off), workspace=ws).cpu().numpy()
    assert mmv.last_async_status(ws) == 0
    assert_fp(got, want, a, f"bf16 seg-sum n={n} p={p}")
    k = torch.zeros(1, dtype=torch.int64, device="cuda")
    ws = mmv.alloc_workspace(mmv.OP_SEG_SUM, mmv.BF16_TO_F32, mmv.SEG_FLAGS_U8, n)
    gotf = mmv.seg_sum(xd, fd, num_segments=k, workspace=ws)
    assert mmv.last_async_status(ws) == 0 and int(k.item()) == off.shape[0] - 1
    wantf, af = oracle.seg_sum_flags_bf16(xb, f)
    assert_fp(gotf[:int(k.item())].cpu().numpy(), wantf, af, f"bf16 flag-form seg-sum n={n} p={p}")


def test_bf16_values_beyond_the_fp16_range(mmv):
    # magnitudes that fp16 cannot hold (up to 1e30 and down to 1e-30), one magnitude per segment
    rng = np.random.default_rng(5)
    nseg = 3000
    lens = rng.integers(1, 200, nseg)
    off = gen.offsets_from_lengths(lens)
    n = int(off[-1])
    scale = np.repeat(10.0 ** rng.integers(-30, 31, nseg).astype(np.float64), lens)
    xb = gen.bf16_bits_of((rng.standard_normal(n) * scale).astype(np.float32))
    f = gen.start_flags_of_offsets(off, n)
    want, a = oracle.seg_scan_bf16(xb, f)
    got = mmv.seg_scan(dev_bf16(xb), dev(f)).cpu().numpy()
    # the bound is relative to the segment's own running sum of magnitudes; what a prefix difference can keep
    # is relative to the magnitudes of its 32-element row, so only segments that dominate their rows are held to it
    ok = np.abs(got - want) <= 2e-3 * a + 1e-6
    big = scale >= np.maximum.accumulate(scale)                        # no larger magnitude before it
    assert ok[big].all()
    assert np.isfinite(got).all()


def test_spmv_tiny_rows_next_to_large_rows(mmv):
    # rows of 1..8 non-zeros whose products are around 1e-3 between rows whose products are around 1e3: the bound
    # is relative to each row's own sum of magnitudes, so a tiny row must not drown in its neighbours' prefixes
    rng = np.random.default_rng(31)
    rows, cols = 50000, 4096
    lens = rng.integers(1, 9, rows)
    rowptr = gen.offsets_from_lengths(lens)
    nnz = int(rowptr[-1])
    col = rng.integers(0, cols, nnz).astype(np.int32)
    big = np.repeat(rng.integers(0, 2, rows).astype(bool), lens)
    val = (rng.standard_normal(nnz) * np.where(big, 1000.0, 1e-3)).astype(np.float16)
    x = (0.5 + rng.random(cols)).astype(np.float32)                  # magnitudes of order 1: the products keep the contrast
    want, a = oracle.spmv_csr(rowptr, col, val, x)
    assert_fp(spmv(mmv, rowptr, col, val, x), want, a, "tiny rows next to large rows")


# ---------------------------------------------------------------------------
# robustness
# ---------------------------------------------------------------------------
def test_bad_column_indices_are_reported_not_dereferenced(mmv):
    rowptr, col, val, xv = gen.config4(rows=4096)
    col = col.copy()
    col[[5, col.shape[0] // 2, col.shape[0] - 1]] = [-7, xv.shape[0], 2 ** 31 - 1]
    ws = mmv.alloc_workspace(mmv.OP_SPMV_CSR, mmv.F16_TO_F32, mmv.SEG_OFFSETS_I32, val.shape[0], 4096)
    mmv.spmv_csr(dev(rowptr), dev(col), dev(val), dev(xv), workspace=ws)
    assert mmv.last_async_status(ws) == 1          # MMV_ERR_INVALID_ARG, and the context is still usable
    ok = col.copy()
    ok[[5, col.shape[0] // 2, col.shape[0] - 1]] = 0
    y = mmv.spmv_csr(dev(rowptr), dev(ok), dev(val), dev(xv), workspace=ws)
    assert mmv.last_async_status(ws) == 0
    want, a = oracle.spmv_csr(rowptr, ok, val, xv)
    assert_fp(y.cpu().numpy(), want, a, "SpMV after a rejected call")


def test_bad_offsets_are_reported_not_trapped(mmv):
    n = 50000
    x = dev(np.ones(n, np.int8))
    off = dev(np.asarray([0, 30000, 20000, n], np.int32))
    ws = mmv.alloc_workspace(mmv.OP_SEG_SUM, mmv.I8_TO_I32, mmv.SEG_OFFSETS_I32, n, 3)
    mmv.seg_sum(x, off, workspace=ws)
    assert mmv.last_async_status(ws) == 4
    ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN, mmv.I8_TO_I32, mmv.SEG_OFFSETS_I32, n, 3)
    mmv.seg_scan(x, off, workspace=ws)
    assert mmv.last_async_status(ws) == 4
    # the context is still usable
    f = np.zeros(n, np.uint8)
    assert np.array_equal(scan_i8(mmv, np.ones(n, np.int8), f), np.arange(1, n + 1))


def test_lookback_wait_gives_up_with_a_status(mmv):
    # one span never publishes its carry: its successors must time out, report it and return
    n = 40 * TILE
    x, f = dev(np.ones(n, np.int8)), dev(np.zeros(n, np.uint8))
    ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN, mmv.I8_TO_I32, mmv.SEG_FLAGS_U8, n)
    try:
        mmv.debug_configure(20_000_000, 17)           # 20 ms budget, span 17 stays silent
        mmv.seg_scan(x, f, workspace=ws)
        assert mmv.last_async_status(ws) == 5
    finally:
        mmv.debug_configure(0, -1)
    out = mmv.seg_scan(x, f, workspace=ws)            # and the next call works
    assert mmv.last_async_status(ws) == 0
    assert np.array_equal(out.cpu().numpy(), np.arange(1, n + 1))


def test_minmax_lookback_wait_gives_up_with_a_status(mmv):
    # the same for the running maximum: the run that holds span 17 stays silent, the runs behind it give up
    n = 40 * MM_TILE
    x = np.arange(n, dtype=np.int64) % 100
    x = dev(x.astype(np.int8))
    ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN_MINMAX, mmv.I8_TO_I32, mmv.SEG_FLAGS_U8, n)
    try:
        mmv.debug_configure(20_000_000, 17)
        mmv.seg_scan_minmax(x, None, workspace=ws)
        assert mmv.last_async_status(ws) == 5
    finally:
        mmv.debug_configure(0, -1)
    out = mmv.seg_scan_minmax(x, None, workspace=ws)   # and the next call works
    assert mmv.last_async_status(ws) == 0
    assert np.array_equal(out.cpu().numpy(), np.minimum(np.arange(n), 99))


# ---------------------------------------------------------------------------
# the calls only enqueue a memset and kernels on the given stream: they can be captured in a CUDA
# graph and replayed (the first call on a device, which sets the kernels' attributes, comes before)
# ---------------------------------------------------------------------------
def test_calls_that_overlap_on_two_streams(mmv):
    # The tiled kernels hand out their tiles in a fixed order and need every CTA of their grid resident; they are
    # launched cooperatively, so two calls that overlap in time on two streams (each with a workspace of its own)
    # run one after the other instead of sharing the SMs and waiting for tiles whose CTAs never started.  A 200 ms
    # wait budget turns any such stall into MMV_ERR_TIMEOUT quickly; what is promised is that none occurs.
    mmv.debug_configure(200_000_000, -1)
    try:
        n = (1 << 27) + 4321
        rng = np.random.default_rng(99)
        xs = [rng.integers(-128, 128, n).astype(np.int8) for _ in range(2)]
        fs = [(rng.random(n) < p).astype(np.uint8) for p in (1e-5, 0.02)]
        want = [oracle.seg_scan_i8(x, f) for x, f in zip(xs, fs)]
        xd, fd = [dev(x) for x in xs], [dev(f) for f in fs]
        outs = [torch.empty(n, dtype=torch.int32, device="cuda") for _ in range(2)]
        wss = [mmv.alloc_workspace(mmv.OP_SEG_SCAN, mmv.I8_TO_I32, mmv.SEG_FLAGS_U8, n) for _ in range(2)]
        streams = [torch.cuda.Stream(), torch.cuda.Stream()]
        torch.cuda.synchronize()
        for _ in range(6):                               # back to back, no host synchronisation in between
            for i in range(2):
                mmv.seg_scan(xd[i], fd[i], out=outs[i], workspace=wss[i], stream=streams[i])
        for i in range(2):
            assert mmv.last_async_status(wss[i], streams[i]) == 0
            assert np.array_equal(outs[i].cpu().numpy(), want[i])
        # a scan beside a segmented sum
        x2, off = gen.config2(1 << 24, max_len=300)
        nseg = off.shape[0] - 1
        x2d, offd = dev(x2), dev(off)
        out2 = torch.empty(nseg, dtype=torch.float32, device="cuda")
        ws2 = mmv.alloc_workspace(mmv.OP_SEG_SUM, mmv.F16_TO_F32, mmv.SEG_OFFSETS_I32, x2.shape[0], nseg)
        torch.cuda.synchronize()
        for _ in range(6):
            mmv.seg_scan(xd[0], fd[0], out=outs[0], workspace=wss[0], stream=streams[0])
            mmv.seg_sum(x2d, offd, out=out2, workspace=ws2, stream=streams[1])
        assert mmv.last_async_status(wss[0], streams[0]) == 0
        assert mmv.last_async_status(ws2, streams[1]) == 0
        assert np.array_equal(outs[0].cpu().numpy(), want[0])
        w2, a2 = oracle.seg_sum_csr_f16(x2, off)
        assert_fp(out2.cpu().numpy(), w2, a2, "segmented sum beside a scan")
    finally:
        mmv.debug_configure(0, -1)


def test_calls_replay_from_a_cuda_graph(mmv):
    rng = np.random.default_rng(5)
    n = 3 * TILE + 4001
    x = rng.integers(-128, 128, n).astype(np.int8)
    f = (rng.random(n) < 0.01).astype(np.uint8)
    off = gen.offsets_from_lengths(rng.integers(0, 700, 400))
    xs = rng.integers(-128, 128, int(off[-1])).astype(np.int8)
    rowptr, col, val, xv = gen.config4(rows=3000, empty_fraction=0.1)
    xd, fd, od_, xsd = dev(x), dev(f), dev(off), dev(xs)
    rd, cd, vd, xvd = dev(rowptr), dev(col), dev(val), dev(xv)
    ws1 = mmv.alloc_workspace(mmv.OP_SEG_SCAN, mmv.I8_TO_I32, mmv.SEG_FLAGS_U8, n)
    ws2 = mmv.alloc_workspace(mmv.OP_SEG_SUM, mmv.I8_TO_I32, mmv.SEG_OFFSETS_I32, xs.shape[0], off.shape[0] - 1)
    ws3 = mmv.alloc_workspace(mmv.OP_SPMV_CSR, mmv.F16_TO_F32, mmv.SEG_OFFSETS_I32, val.shape[0], 3000)
    o1 = torch.zeros(n, dtype=torch.int32, device="cuda")
    o2 = torch.zeros(off.shape[0] - 1, dtype=torch.int32, device="cuda")
    o3 = torch.zeros(3000, dtype=torch.float32, device="cuda")
    ws4 = mmv.alloc_workspace(mmv.OP_SEG_SCAN_MINMAX, mmv.I8_TO_I32, mmv.SEG_FLAGS_U8, n)
    ws5 = mmv.alloc_workspace(mmv.OP_SEG_SCAN_WIDE, mmv.I8_TO_I32, mmv.SEG_FLAGS_U8, n)
    ws6 = mmv.alloc_workspace(mmv.OP_COMPRESS, mmv.I8_TO_I32, mmv.SEG_FLAGS_U8, n)
    o4 = torch.zeros(n, dtype=torch.int32, device="cuda")
    o5 = torch.zeros(n, dtype=torch.int64, device="cuda")
    o6 = torch.zeros(n, dtype=torch.int8, device="cuda")
    k6 = torch.zeros(1, dtype=torch.int64, device="cuda")

    def calls():
        mmv.seg_scan(xd, fd, out=o1, workspace=ws1)
        mmv.seg_sum(xsd, od_, out=o2, workspace=ws2)
        mmv.spmv_csr(rd, cd, vd, xvd, y=o3, workspace=ws3)
        mmv.seg_scan_minmax(xd, fd, want_min=True, out=o4, workspace=ws4)
        mmv.seg_scan_wide(xd, fd, out=o5, workspace=ws5)
        mmv.compress(xd, fd, out=o6, count=k6, workspace=ws6)

    calls()                                   # warm-up outside the capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        calls()
    for buf in (o1, o2, o3, o4, o5, o6, k6):
        buf.zero_()
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    assert mmv.last_async_status(ws1) == 0 and mmv.last_async_status(ws2) == 0 and mmv.last_async_status(ws3) == 0
    assert np.array_equal(o1.cpu().numpy(), oracle.seg_scan_i8(x, f))
    assert np.array_equal(o2.cpu().numpy(), oracle.seg_sum_csr_i8(xs, off))
    want, a = oracle.spmv_csr(rowptr, col, val, xv)
    assert_fp(o3.cpu().numpy(), want, a, "SpMV replayed from a graph")
    assert mmv.last_async_status(ws4) == 0 and mmv.last_async_status(ws5) == 0
    assert np.array_equal(o4.cpu().numpy(), oracle.seg_scan_minmax_i8(x, f, True))
    assert np.array_equal(o5.cpu().numpy(), oracle.seg_scan_i8_wide(x, f))
    kept = oracle.compress(x, f)
    assert int(k6.item()) == kept.shape[0] and np.array_equal(o6[:kept.shape[0]].cpu().numpy(), kept)


# ---------------------------------------------------------------------------
# one vector scanned as contiguous shards (the multi-GPU path, all shards on this GPU)
# ---------------------------------------------------------------------------
def scan_in_shards(mmv, x, f, cuts):
    """x/f cut at `cuts`: every shard is scanned by itself, the 16-byte records are gathered into one buffer
    (here by device copies; across GPUs by one all-gather) and every shard adds its carry."""
    n = x.shape[0]
    edges = [0] + list(cuts) + [n]
    world = len(edges) - 1
    odt = torch.int32 if x.dtype == np.int8 else torch.float32
    xd = dev_bf16(x) if x.dtype == np.uint16 else dev(x)
    fd = dev(f)
    out = torch.full((n + 64,), -777, dtype=odt, device="cuda")
    gathered = torch.zeros(2 * world, dtype=torch.int64, device="cuda")
    mine = [torch.zeros(2, dtype=torch.int64, device="cuda") for _ in range(world)]
    wss = []
    for r in range(world):
        a, b = edges[r], edges[r + 1]
        ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN, mmv.F16_TO_F32, mmv.SEG_FLAGS_U8, max(1, b - a))
        wss.append(ws)
        mmv.seg_scan_shard(xd[a:b], fd[a:b], r == 0, out[a:b], mine[r], ws)
    for r in range(world):
        gathered[2 * r:2 * r + 2] = mine[r]                       # the all-gather
    for r in range(world):
        a, b = edges[r], edges[r + 1]
        mmv.seg_scan_shard_finish(gathered, r, world, out[a:b], xd.dtype)
    for ws in wss:
        assert mmv.last_async_status(ws) == 0
    got = out.cpu().numpy()
    assert (got[n:] == -777).all()
    return got[:n], gathered.cpu().numpy().reshape(world, 2)


@pytest.mark.parametrize("p", [0.0, 1e-5, 1e-3, 0.3])
def test_scan_in_four_shards_matches_the_whole_vector(mmv, p):
    rng = np.random.default_rng(int(p * 1e6) + 3)
    n = 37 * TILE + 4321
    cuts = [8 * TILE, 8 * TILE + 16 * 1000, 30 * TILE + 16]        # shard edges must keep 16-byte alignment of x, f, out
    f = (rng.random(n) < p).astype(np.uint8)
    f[cuts[1]] = 1                                                  # one shard begins with a start ...
    f[cuts[2]] = 0                                                  # ... another continues the segment in front of it
    xi = rng.integers(-128, 128, n).astype(np.int8)
    got, rec = scan_in_shards(mmv, xi, f, cuts)
    assert np.array_equal(got, oracle.seg_scan_i8(xi, f))
    # the records: first start of every shard (flag byte 0 of shard 0 is not consulted: element 0 starts)
    edges = [0] + cuts + [n]
    for r in range(4):
        fl = f[edges[r]:edges[r + 1]].copy()
        if r == 0:
            fl[0] = 1
        nz = np.flatnonzero(fl)
        assert rec[r, 1] == (nz[0] if nz.size else fl.shape[0])
        assert (rec[r, 0] >> 32) == (1 if nz.size else 0)
    xf = rng.uniform(-1, 1, n).astype(np.float16)
    z, a = oracle.seg_scan_f16(xf, f)
    assert_fp(scan_in_shards(mmv, xf, f, cuts)[0], z, a, f"fp16 in shards, p={p}")
    xb = gen.bf16_normal(12, n)
    zb, ab = oracle.seg_scan_bf16(xb, f)
    assert_fp(scan_in_shards(mmv, xb, f, cuts)[0], zb, ab, f"bf16 in shards, p={p}")


def test_scan_in_shards_edges(mmv):
    # shards shorter than a tile, a single shard, a shard without any start between two that have one, and the
    # flag-free call (no flag vector at all)
    rng = np.random.default_rng(8)
    n = 5 * TILE + 48
    xi = rng.integers(-128, 128, n).astype(np.int8)
    f = np.zeros(n, np.uint8)
    f[[100, 4 * TILE + 7]] = 1
    for cuts in ([], [16], [16, 32, 48], [TILE, 3 * TILE], [n - 16]):
        got, _ = scan_in_shards(mmv, xi, f, cuts)
        assert np.array_equal(got, oracle.seg_scan_i8(xi, f)), cuts
    world, m = 3, TILE + 160
    x3 = torch.from_numpy(xi[:world * m]).cuda()
    out = torch.empty(world * m, dtype=torch.int32, device="cuda")
    gathered = torch.zeros(2 * world, dtype=torch.int64, device="cuda")
    for r in range(world):
        ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN, mmv.I8_TO_I32, mmv.SEG_FLAGS_U8, m)
        mmv.seg_scan_shard(x3[r * m:(r + 1) * m], None, r == 0, out[r * m:(r + 1) * m], gathered[2 * r:2 * r + 2], ws)
    for r in range(world):
        mmv.seg_scan_shard_finish(gathered, r, world, out[r * m:(r + 1) * m], torch.int8)
    assert np.array_equal(out.cpu().numpy(), oracle.seg_scan_i8(xi[:world * m], np.zeros(world * m, np.uint8)))


# ---------------------------------------------------------------------------
# the narrow-tile shape of the floating-point scan (chosen by the library where starts are rare) on every density
# ---------------------------------------------------------------------------
def test_scan_narrow_shape_is_correct_for_every_flag_vector(mmv):
    # forced for all calls below: pieces that hold a start fetch their rows from memory instead of identity columns
    mmv.debug_force_scan_shape(2)
    try:
        for n in (1, 33, 1025, 4097, TILE - 1, TILE + 1, 5 * TILE + 4099, 100_003):
            test_scan_f16_sizes(mmv, n)
        test_scan_flag_positions_around_row_and_tile_edges(mmv)
        test_scan_closed_forms(mmv)
        test_scan_with_offsets(mmv)
        test_scan_tiny_segments_next_to_large_values(mmv)
        test_scan_mixed_magnitudes_inside_a_segment(mmv)
        for n, p in ((4097, 0.05), (3 * TILE + 4097, 1e-3), (11 * TILE + 777, 0.5), (11 * TILE + 777, 1.0)):
            test_exclusive_scan(mmv, n, p)
        for n, p in ((33, 1.0), (7 * TILE + 1234, 1e-3), (7 * TILE + 1234, 0.1)):
            test_bf16_scan_and_sum(mmv, n, p)
        test_bf16_values_beyond_the_fp16_range(mmv)
        test_scan_in_four_shards_matches_the_whole_vector(mmv, 1e-5)
        test_lookback_wait_gives_up_with_a_status(mmv)
        # many tiles per warpgroup, few starts: the case the shape is for
        rng = np.random.default_rng(4)
        n = 300 * TILE + 77
        x = rng.uniform(-1, 1, n).astype(np.float16)
        for p in (0.0, 1e-6, 1e-4):
            f = (rng.random(n) < p).astype(np.uint8)
            z, a = oracle.seg_scan_f16(x, f)
            assert_fp(scan_f16(mmv, x, f), z, a, f"narrow shape, p={p}")
    finally:
        mmv.debug_force_scan_shape(-1)


# ---------------------------------------------------------------------------
# element-wise integer product through the segmented sum (Corollary 4.5)
# ---------------------------------------------------------------------------
def test_mult_i8_is_exact(mmv):
    v = np.arange(-128, 128, dtype=np.int64)
    xs, ys = np.repeat(v, 256).astype(np.int8), np.tile(v, 256).astype(np.int8)          # every pair of int8 values
    got = mmv.mult_i8(dev(xs), dev(ys)).cpu().numpy()
    assert np.array_equal(got, oracle.mult_i8(xs, ys))
    rng = np.random.default_rng(6)
    for n in (1, 7, 511, 513, 2049, 40 * TILE // 8 + 3, 300_001):
        x = rng.integers(-128, 128, n).astype(np.int8)
        y = rng.integers(-128, 128, n).astype(np.int8)
        ws = mmv.alloc_workspace(mmv.OP_MULT, mmv.I8_TO_I32, mmv.SEG_OFFSETS_I32, n)
        buf = torch.full((n + 16,), -777, dtype=torch.int32, device="cuda")
        mmv.mult_i8(dev(x), dev(y), out=buf[:n], workspace=ws)
        assert mmv.last_async_status(ws) == 0
        g = buf.cpu().numpy()
        assert (g[n:] == -777).all()
        assert np.array_equal(g[:n], oracle.mult_i8(x, y)), n
    assert mmv.mult_i8(dev(np.zeros(0, np.int8)), dev(np.zeros(0, np.int8))).numel() == 0
