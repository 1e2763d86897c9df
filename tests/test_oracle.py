"""Pins for the CPU oracle: values the paper prints, closed forms, brute force,
library routines and independent formulations.  No GPU needed."""
import itertools
from fractions import Fraction

import numpy as np
import pytest

import mmv_inputs as gen
import oracle
from conftest import load_golden


def f16(a):
    return np.asarray(a, np.float32).astype(np.float16)


def u8(a):
    return np.asarray(a, np.uint8)


# --------------------------------------------------------------------------
# brute force that shares nothing with the recurrence: z(i) = sum x[start(i)..i]
# --------------------------------------------------------------------------
def brute_scan(x, f):
    n = len(x)
    z = []
    for i in range(n):
        s = i
        while s > 0 and f[s] == 0:
            s -= 1
        z.append(sum(x[s:i + 1]))
    return z


def brute_sums(x, f):
    z = brute_scan(x, f)
    n = len(x)
    return [z[i] for i in range(n) if i == n - 1 or f[i + 1] != 0]


def wrap32(v):
    return int(np.int64(v).astype(np.int32)) if -2 ** 63 <= v < 2 ** 63 else None


# --------------------------------------------------------------------------
# the paper's worked example (Section 2)
# --------------------------------------------------------------------------
def test_paper_worked_example():
    g = load_golden("sec2_worked_example.txt")
    x, f = g["x"], g["f"]
    z, a = oracle.seg_scan_f16(f16(x), u8(f))
    assert z.tolist() == g["seg_scan"]
    assert a.tolist() == g["seg_scan"]          # all values positive: a == z
    zi = oracle.seg_scan_i8(np.asarray(x, np.int8), u8(f))
    assert zi.tolist() == g["seg_scan"]
    s, _ = oracle.seg_sum_flags_f16(f16(x), u8(f))
    assert s.tolist() == g["seg_sum"]
    assert oracle.seg_sum_flags_i8(np.asarray(x, np.int8), u8(f)).tolist() == g["seg_sum"]
    # COMPRESS(x, f) of the same example keeps x where f is set
    assert [xi for xi, fi in zip(x, f) if fi] == g["compress_x_f"]
    # the same segments as CSR offsets
    off = np.asarray([0, 2, 5, 8], np.int32)
    assert oracle.seg_sum_csr_i8(np.asarray(x, np.int8), off).tolist() == g["seg_sum"]
    assert oracle.seg_sum_csr_f16(f16(x), off)[0].tolist() == g["seg_sum"]
    assert oracle.flags_from_offsets(off, 8).tolist() == f


def test_hand_worked_n16():
    g = load_golden("hand_worked_n16_s4.txt")
    x, f = g["x"], g["f"]
    assert oracle.seg_scan_i8(np.asarray(x, np.int8), u8(f)).tolist() == g["seg_scan"]
    assert oracle.seg_scan_f16(f16(x), u8(f))[0].tolist() == g["seg_scan"]
    assert oracle.seg_sum_flags_i8(np.asarray(x, np.int8), u8(f)).tolist() == g["seg_sum"]
    # the fixture's speculative block scans are plain per-block prefix sums
    assert np.cumsum(np.asarray(x).reshape(4, 4), axis=1).ravel().tolist() == g["block_scan"]
    assert np.cumsum(np.asarray(f).reshape(4, 4), axis=1).ravel().tolist() == g["block_flag_scan"]


def test_first_flag_is_ignored():
    # index 0 always opens a segment, whatever f(0) says (Eq. 1: "i = 0 or f(i) = 1")
    x, f = [1, 2, 3, 4], [0, 0, 1, 0]
    assert oracle.seg_scan_i8(np.asarray(x, np.int8), u8(f)).tolist() == [1, 3, 3, 7]
    assert oracle.seg_sum_flags_i8(np.asarray(x, np.int8), u8(f)).tolist() == [3, 7]
    f1 = [1, 0, 1, 0]
    assert oracle.seg_scan_i8(np.asarray(x, np.int8), u8(f1)).tolist() == [1, 3, 3, 7]


def test_any_nonzero_flag_byte_starts_a_segment():
    x = np.asarray([1, 1, 1, 1, 1], np.int8)
    f = u8([1, 0, 200, 0, 7])
    assert oracle.seg_scan_i8(x, f).tolist() == [1, 2, 1, 2, 1]


def test_csr_examples():
    g = load_golden("csr_examples.txt")
    x = np.asarray(g["sum_x"], np.int8)
    off = np.asarray(g["sum_off"], np.int32)
    assert oracle.seg_sum_csr_i8(x, off).tolist() == g["sum_out"]
    out, a = oracle.seg_sum_csr_f16(f16(g["sum_x"]), off)
    assert out.tolist() == g["sum_out"] and a.tolist() == g["sum_out"]
    y, a = oracle.spmv_csr(np.asarray(g["spmv_rowptr"], np.int32), np.asarray(g["spmv_col"], np.int32),
                           f16(g["spmv_val"]), np.asarray(g["spmv_x"], np.float32))
    assert y.tolist() == g["spmv_y"] and a.tolist() == g["spmv_y"]


# --------------------------------------------------------------------------
# closed forms
# --------------------------------------------------------------------------
@pytest.mark.parametrize("n", [1, 2, 7, 128, 1000, 4099])
def test_all_ones_gives_position_in_segment(n):
    rng = np.random.default_rng(n)
    f = (rng.random(n) < 0.1).astype(np.uint8)
    start = np.maximum.accumulate(np.where((f != 0) | (np.arange(n) == 0), np.arange(n), 0))
    want = np.arange(n) - start + 1
    z = oracle.seg_scan_i8(np.ones(n, np.int8), f)
    assert np.array_equal(z, want)
    zf, a = oracle.seg_scan_f16(np.ones(n, np.float16), f)
    assert np.array_equal(zf, want) and np.array_equal(a, want)


@pytest.mark.parametrize("n", [1, 5, 333])
def test_all_flags_is_identity(n):
    rng = np.random.default_rng(n + 1)
    x = rng.integers(-128, 128, n).astype(np.int8)
    f = np.ones(n, np.uint8)
    assert np.array_equal(oracle.seg_scan_i8(x, f), x.astype(np.int32))
    assert np.array_equal(oracle.seg_sum_flags_i8(x, f), x.astype(np.int32))
    xf = rng.standard_normal(n).astype(np.float16)
    z, a = oracle.seg_scan_f16(xf, f)
    assert np.array_equal(z, xf.astype(np.float64)) and np.array_equal(a, np.abs(xf.astype(np.float64)))
    s, _ = oracle.seg_sum_flags_f16(xf, f)
    assert np.array_equal(s, xf.astype(np.float64))


@pytest.mark.parametrize("n", [1, 6, 1025])
def test_no_flags_is_plain_prefix_sum(n):
    rng = np.random.default_rng(n + 2)
    x = rng.integers(-128, 128, n).astype(np.int8)
    f = np.zeros(n, np.uint8)
    assert np.array_equal(oracle.seg_scan_i8(x, f), np.cumsum(x.astype(np.int64)).astype(np.int32))
    assert oracle.seg_sum_flags_i8(x, f).tolist() == [int(x.astype(np.int64).sum())]
    xf = rng.standard_normal(n).astype(np.float16)
    z, a = oracle.seg_scan_f16(xf, f)
    np.testing.assert_allclose(z, np.cumsum(xf.astype(np.float64)), rtol=0, atol=1e-12)
    np.testing.assert_allclose(a, np.cumsum(np.abs(xf.astype(np.float64))), rtol=0, atol=1e-12)


def test_triangular_numbers():
    n = 100
    x = np.arange(1, n + 1).astype(np.int8)
    z = oracle.seg_scan_i8(x, np.zeros(n, np.uint8))
    i = np.arange(n)
    assert np.array_equal(z, (i + 1) * (i + 2) // 2)


def test_cycle_1_2_3():
    n = 60
    f = np.tile(u8([1, 1, 0, 1, 0, 0]), n // 6)
    z = oracle.seg_scan_i8(np.ones(n, np.int8), f)
    assert z.tolist() == [1, 1, 2, 1, 2, 3] * (n // 6)
    assert oracle.seg_sum_flags_i8(np.ones(n, np.int8), f).tolist() == [1, 2, 3] * (n // 6)


def test_int_wraps_mod_2_32():
    # 2^25 values of -128 with no flags: the exact total is -2^32, which wraps to 0
    n = 1 << 25
    x = np.full(n, -128, np.int8)
    z = oracle.seg_scan_i8(x, np.zeros(n, np.uint8))
    assert z[-1] == 0
    k = (1 << 24) - 1                       # exact prefix -(2^24)*128 = -2^31: still representable
    assert z[k] == -2 ** 31
    assert z[k + 1] == 2 ** 31 - 128        # -2^31 - 128 wraps
    assert oracle.seg_sum_flags_i8(x, np.zeros(n, np.uint8)).tolist() == [0]
    assert oracle.seg_sum_csr_i8(x, np.asarray([0, n], np.int32)).tolist() == [0]


def test_half_decode_matches_numpy_for_every_bit_pattern():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    want = bits.view(np.float16).astype(np.float64)
    # drive the decoder through the scan with every element its own segment
    z, a = oracle.seg_scan_f16(bits, np.ones(65536, np.uint8))
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(z), nan)
    assert np.array_equal(z[~nan], want[~nan])
    assert np.array_equal(a[~nan], np.abs(want[~nan]))
    assert oracle.half_to_double(0x3C00) == 1.0 and oracle.half_to_double(0x0001) == 2.0 ** -24
    assert oracle.half_to_double(0xC000) == -2.0 and oracle.half_to_double(0x7BFF) == 65504.0


# --------------------------------------------------------------------------
# brute force
# --------------------------------------------------------------------------
def test_exhaustive_small_n_all_flag_vectors():
    rng = np.random.default_rng(7)
    for n in range(1, 11):
        x = rng.integers(-9, 10, n).tolist()
        for bits in itertools.product([0, 1], repeat=n):
            want = brute_scan(x, bits)
            got = oracle.seg_scan_i8(np.asarray(x, np.int8), u8(bits))
            assert got.tolist() == want, (x, bits)
            assert oracle.seg_sum_flags_i8(np.asarray(x, np.int8), u8(bits)).tolist() == brute_sums(x, bits)
    n = 12
    x = rng.integers(-9, 10, n).tolist()
    for bits in itertools.product([0, 1], repeat=n):
        assert oracle.seg_scan_f16(f16(x), u8(bits))[0].tolist() == brute_scan(x, bits)


def test_random_brute_force_fp16_exact_rationals():
    rng = np.random.default_rng(11)
    for trial in range(60):
        n = int(rng.integers(1, 65))
        x = rng.standard_normal(n).astype(np.float16)
        f = (rng.random(n) < rng.choice([0.05, 0.3, 0.7])).astype(np.uint8)
        xq = [Fraction(float(v)) for v in x]
        want = brute_scan(xq, f.tolist())
        want_a = brute_scan([abs(v) for v in xq], f.tolist())
        z, a = oracle.seg_scan_f16(x, f)
        for i in range(n):
            assert abs(Fraction(float(z[i])) - want[i]) <= Fraction(1, 10 ** 12)
            assert abs(Fraction(float(a[i])) - want_a[i]) <= Fraction(1, 10 ** 12)
        s, sa = oracle.seg_sum_flags_f16(x, f)
        ws = brute_sums(xq, f.tolist())
        assert len(s) == len(ws) == 1 + int(np.count_nonzero(f[1:]))
        for got, w in zip(s, ws):
            assert abs(Fraction(float(got)) - w) <= Fraction(1, 10 ** 12)


def test_random_brute_force_int8():
    rng = np.random.default_rng(13)
    for trial in range(200):
        n = int(rng.integers(1, 65))
        x = rng.integers(-128, 128, n).astype(np.int8)
        f = (rng.random(n) < rng.choice([0.02, 0.25, 0.8])).astype(np.uint8)
        assert oracle.seg_scan_i8(x, f).tolist() == brute_scan(x.astype(int).tolist(), f.tolist())
        assert oracle.seg_sum_flags_i8(x, f).tolist() == brute_sums(x.astype(int).tolist(), f.tolist())


# --------------------------------------------------------------------------
# library routines
# --------------------------------------------------------------------------
def test_csr_sum_against_reduceat_and_python_sum():
    rng = np.random.default_rng(17)
    for trial in range(30):
        nseg = int(rng.integers(1, 40))
        lens = rng.integers(0, 9, nseg)
        off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
        n = int(off[-1])
        x = rng.integers(-128, 128, n).astype(np.int8)
        want = [int(x[off[r]:off[r + 1]].astype(np.int64).sum()) for r in range(nseg)]
        assert oracle.seg_sum_csr_i8(x, off).tolist() == want
        nz = np.flatnonzero(lens > 0)
        if n and nz.size:
            ra = np.add.reduceat(x.astype(np.int64), off[:-1][nz])
            assert np.array_equal(oracle.seg_sum_csr_i8(x, off)[nz], ra)
        xf = rng.standard_normal(n).astype(np.float16)
        out, a = oracle.seg_sum_csr_f16(xf, off)
        for r in range(nseg):
            seg = xf[off[r]:off[r + 1]].astype(np.float64)
            assert abs(out[r] - seg.sum()) <= 1e-12 and abs(a[r] - np.abs(seg).sum()) <= 1e-12
            if lens[r] == 0:
                assert out[r] == 0.0 and a[r] == 0.0


def test_spmv_against_scipy():
    sp = pytest.importorskip("scipy.sparse")
    rng = np.random.default_rng(19)
    rows, cols = 57, 41
    lens = rng.integers(0, 12, rows)
    lens[[0, 5, rows - 1]] = 0
    rowptr = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    nnz = int(rowptr[-1])
    col = rng.integers(0, cols, nnz).astype(np.int32)
    val = rng.uniform(-1, 1, nnz).astype(np.float16)
    x = rng.standard_normal(cols).astype(np.float32)
    A = sp.csr_matrix((val.astype(np.float64), col.copy(), rowptr.copy()), shape=(rows, cols))
    want = A @ x.astype(np.float64)
    Aabs = sp.csr_matrix((np.abs(val.astype(np.float64)), col.copy(), rowptr.copy()), shape=(rows, cols))
    want_a = Aabs @ np.abs(x.astype(np.float64))
    y, a = oracle.spmv_csr(rowptr, col, val, x)
    np.testing.assert_allclose(y, want, rtol=0, atol=1e-12)
    np.testing.assert_allclose(a, want_a, rtol=0, atol=1e-12)
    assert y[0] == 0.0 and y[5] == 0.0 and y[rows - 1] == 0.0


# --------------------------------------------------------------------------
# independent formulations from the paper (integers: exact)
# --------------------------------------------------------------------------
def scd(x, f):
    """Algorithm 4.2: DIFF(COMPRESS(SCAN(x), f^-)), f^- = f shifted left with 1 appended."""
    xs = np.cumsum(np.asarray(x, np.int64))
    fm = np.concatenate([np.asarray(f[1:], np.uint8), [1]])
    z = xs[fm != 0]
    return np.diff(np.concatenate([[0], z]))


def sscr(x, f):
    """Algorithm 4.3: subtract from every segment the speculative scan value at the
    end of the previous segment.  With f(0) counted as a start the k-th segment
    (k = flag prefix count) subtracts w(k-2); the printed index is one off."""
    f = np.asarray(f, np.uint8).copy()
    f[0] = 1
    xs = np.cumsum(np.asarray(x, np.int64))
    fs = np.cumsum(f.astype(np.int64))
    fm = np.concatenate([f[1:], [1]])
    w = xs[fm != 0]
    z = xs.copy()
    for idx in range(len(w)):
        z = z - (fs == idx + 2) * w[idx]
    return z


def block_recursive(x, f, s):
    """The six-step block-recursive recipe of Section 4.2 (Algorithm A.1), with the
    carry added only to positions strictly after the carry source."""
    x = np.asarray(x, np.int64)
    f = np.asarray(f, np.uint8).copy()
    n = len(x)
    f[0] = 1
    nb = -(-n // s)
    xp = np.zeros(nb * s, np.int64)
    fp = np.zeros(nb * s, np.uint8)
    xp[:n], fp[:n] = x, f
    X, F = xp.reshape(nb, s), fp.reshape(nb, s)
    # steps 1-2: speculative block scans, then revert (Lemma A.1): subtract the
    # speculative value just before the start of the element's segment
    Xb, Fb = np.cumsum(X, axis=1), np.cumsum(F, axis=1)
    Z = Xb.copy()
    for b in range(nb):
        for j in range(s):
            for i in range(j):
                if Fb[b, i] != Fb[b, i + 1] and Fb[b, j] == Fb[b, i + 1]:
                    Z[b, j] = Xb[b, j] - Xb[b, i]
    if nb == 1:
        return Z.ravel()[:n]
    # steps 3-5: block lasts, OR of flags, recurse
    xs_, fs_ = Z[:, s - 1].copy(), (Fb[:, s - 1] != 0).astype(np.uint8)
    zs = block_recursive(xs_, fs_, s)
    # step 6: add the previous block's last value to the first segment of each block
    for b in range(1, nb):
        for j in range(s):
            if Fb[b, j] == 0:
                Z[b, j] += zs[b - 1]
    return Z.ravel()[:n]


def test_paper_formulations_agree_with_the_definition():
    rng = np.random.default_rng(23)
    for trial in range(150):
        n = int(rng.integers(1, 100))
        x = rng.integers(-20, 21, n).astype(np.int8)
        f = (rng.random(n) < rng.choice([0.03, 0.2, 0.6])).astype(np.uint8)
        z = oracle.seg_scan_i8(x, f).astype(np.int64)
        assert np.array_equal(sscr(x, f), z)
        assert np.array_equal(scd(x, f), oracle.seg_sum_flags_i8(x, f).astype(np.int64))
        for s in (2, 3, 4, 8):
            assert np.array_equal(block_recursive(x, f, s), z), (n, s)


# --------------------------------------------------------------------------
# invariants
# --------------------------------------------------------------------------
def test_invariants_and_concatenation():
    rng = np.random.default_rng(29)
    n = 5000
    x = rng.integers(-128, 128, n).astype(np.int8)
    f = (rng.random(n) < 0.01).astype(np.uint8)
    z = oracle.seg_scan_i8(x, f).astype(np.int64)
    d = np.diff(z)
    cont = f[1:] == 0
    assert np.array_equal(d[cont], x[1:][cont].astype(np.int64))
    assert np.array_equal(z[1:][~cont], x[1:][~cont].astype(np.int64))
    assert int(oracle.seg_sum_flags_i8(x, f).astype(np.int64).sum()) == int(x.astype(np.int64).sum())
    # scanning [a ; b] with a flag on b's first element = scan(a) ++ scan(b)
    k = 1234
    f2 = f.copy()
    f2[k] = 1
    z2 = oracle.seg_scan_i8(x, f2)
    assert np.array_equal(z2[:k], oracle.seg_scan_i8(x[:k], f2[:k]))
    assert np.array_equal(z2[k:], oracle.seg_scan_i8(x[k:], f2[k:]))


def test_streaming_state_equals_whole():
    rng = np.random.default_rng(31)
    n = 10_000
    x = rng.standard_normal(n).astype(np.float16)
    xi = rng.integers(-128, 128, n).astype(np.int8)
    f = (rng.random(n) < 0.002).astype(np.uint8)
    z, a = oracle.seg_scan_f16(x, f)
    zi = oracle.seg_scan_i8(xi, f)
    st, sti = oracle.new_f16_state(), oracle.new_i8_state()
    zs, as_, zis = [], [], []
    for lo in range(0, n, 777):
        zz, aa = oracle.seg_scan_f16(x[lo:lo + 777], f[lo:lo + 777], st)
        zs.append(zz), as_.append(aa)
        zis.append(oracle.seg_scan_i8(xi[lo:lo + 777], f[lo:lo + 777], sti))
    assert np.array_equal(np.concatenate(zs), z) and np.array_equal(np.concatenate(as_), a)
    assert np.array_equal(np.concatenate(zis), zi)


def test_offsets_to_flags_and_scan_by_segments():
    rng = np.random.default_rng(37)
    lens = rng.integers(0, 6, 300)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    n = int(off[-1])
    f = oracle.flags_from_offsets(off, n)
    starts = sorted(set(int(off[r]) for r in range(300) if lens[r] > 0))
    assert np.flatnonzero(f).tolist() == starts
    x = rng.integers(-128, 128, n).astype(np.int8)
    z = oracle.seg_scan_i8(x, f)
    for r in range(300):
        seg = x[off[r]:off[r + 1]].astype(np.int64)
        assert np.array_equal(z[off[r]:off[r + 1]], np.cumsum(seg))
    with pytest.raises(ValueError):
        oracle.flags_from_offsets(np.asarray([0, 3, 2, 5], np.int32), 5)


def test_fp_bound_helper():
    z = np.asarray([1.0, 0.0])
    a = np.asarray([1.0, 0.0])
    ok, ratio, _ = oracle.check_fp(np.asarray([1.0 + 2e-3, 1e-6], np.float64), z, a)
    assert ok and ratio <= 1.0
    ok, ratio, i = oracle.check_fp(np.asarray([1.0, 2e-6], np.float64), z, a)
    assert not ok and i == 1


# --------------------------------------------------------------------------
# exclusive variant: e(i) = sum of the elements of i's segment in front of i
# --------------------------------------------------------------------------
def brute_excl(x, f):
    out = []
    for i in range(len(x)):
        s = i
        while s > 0 and not f[s]:
            s -= 1
        out.append(sum(x[s:i], type(x[0])(0)))
    return out


def test_exclusive_scan_of_the_worked_example_and_exhaustively():
    g = load_golden("sec2_worked_example.txt")
    x, f = g["x"], g["f"]
    # inclusive (2,4,3,6,7,3,4,6) shifted inside each segment: (0,2,0,3,6,0,3,4)
    want = [z - xi for z, xi in zip(g["seg_scan"], x)]
    assert want == [0, 2, 0, 3, 6, 0, 3, 4]
    e, a = oracle.seg_scan_excl_f16(f16(x), u8(f))
    assert e.tolist() == want and a.tolist() == want
    assert oracle.seg_scan_excl_i8(np.asarray(x, np.int8), u8(f)).tolist() == want
    rng = np.random.default_rng(17)
    for n in range(1, 10):
        x = rng.integers(-9, 10, n).tolist()
        for bits in itertools.product([0, 1], repeat=n):
            assert oracle.seg_scan_excl_i8(np.asarray(x, np.int8), u8(bits)).tolist() == brute_excl(x, bits), (x, bits)
            assert oracle.seg_scan_excl_f16(f16(x), u8(bits))[0].tolist() == brute_excl(x, bits)


def test_exclusive_scan_random_and_identities():
    rng = np.random.default_rng(19)
    for trial in range(60):
        n = int(rng.integers(1, 80))
        f = (rng.random(n) < rng.choice([0.03, 0.3, 0.8])).astype(np.uint8)
        x = rng.standard_normal(n).astype(np.float16)
        xq = [Fraction(float(v)) for v in x]
        e, a = oracle.seg_scan_excl_f16(x, f)
        want, want_a = brute_excl(xq, f.tolist()), brute_excl([abs(v) for v in xq], f.tolist())
        for i in range(n):
            assert abs(Fraction(float(e[i])) - want[i]) <= Fraction(1, 10 ** 12)
            assert abs(Fraction(float(a[i])) - want_a[i]) <= Fraction(1, 10 ** 12)
        xi = rng.integers(-128, 128, n).astype(np.int8)
        ei = oracle.seg_scan_excl_i8(xi, f)
        assert ei.tolist() == brute_excl(xi.astype(int).tolist(), f.tolist())
        # exclusive + element = inclusive (exact in integers)
        assert np.array_equal(ei.astype(np.int64) + xi, oracle.seg_scan_i8(xi, f).astype(np.int64))
    # wrap-around: 2^25 elements of 127 pass 2^31
    n = 1 << 25
    e = oracle.seg_scan_excl_i8(np.full(n, 127, np.int8), np.zeros(n, np.uint8))
    for i in (0, 1, (1 << 24) + 5, n - 1):
        assert int(e[i]) == wrap32(127 * i)
    # all flags: zero everywhere; no flags: prefix sums shifted by one
    assert not oracle.seg_scan_excl_i8(np.full(100, 5, np.int8), np.ones(100, np.uint8)).any()
    assert oracle.seg_scan_excl_f16(np.ones(50, np.float16), np.zeros(50, np.uint8))[0].tolist() == list(range(50))


# --------------------------------------------------------------------------
# bfloat16 inputs: exact decode, then the same definitions on double values
# --------------------------------------------------------------------------
def test_bf16_decode_matches_the_float32_bit_pattern_for_every_value():
    bits = np.arange(65536, dtype=np.uint16)
    got = oracle.bf16_to_double(bits)
    with np.errstate(invalid="ignore"):                     # (signalling NaN patterns are among the 65536)
        want = (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)    # bf16 = top half of fp32
    finite = np.isfinite(want)
    assert np.array_equal(got[finite], want[finite])
    assert np.array_equal(np.isnan(got), np.isnan(want)) and np.array_equal(np.isinf(got), np.isinf(want))
    assert np.array_equal(np.signbit(got[~np.isnan(want)]), np.signbit(want[~np.isnan(want)]))
    # rounding of the generator: nearest, ties to even
    x = np.asarray([1.0, 1.00390625, 1.01171875, -2.5, 3.0e38, 1e-40], np.float32)
    assert gen.bf16_bits_of(x).tolist() == [0x3F80, 0x3F80, 0x3F82, 0xC020, 0x7F62, 0x0001]


def test_bf16_definitions_against_brute_force_and_the_fp16_functions():
    rng = np.random.default_rng(23)
    for trial in range(40):
        n = int(rng.integers(1, 70))
        f = (rng.random(n) < rng.choice([0.05, 0.3, 0.8])).astype(np.uint8)
        xb = gen.bf16_bits_of(rng.standard_normal(n).astype(np.float32) * 100)
        xq = [Fraction(float(v)) for v in oracle.bf16_to_double(xb)]
        z, a = oracle.seg_scan_bf16(xb, f)
        e, ea = oracle.seg_scan_bf16(xb, f, exclusive=True)
        want, want_a = brute_scan(xq, f.tolist()), brute_scan([abs(v) for v in xq], f.tolist())
        want_e = brute_excl(xq, f.tolist())
        for i in range(n):
            assert abs(Fraction(float(z[i])) - want[i]) <= Fraction(1, 10 ** 9)
            assert abs(Fraction(float(a[i])) - want_a[i]) <= Fraction(1, 10 ** 9)
            assert abs(Fraction(float(e[i])) - want_e[i]) <= Fraction(1, 10 ** 9)
        s, _ = oracle.seg_sum_flags_bf16(xb, f)
        ws = brute_sums(xq, f.tolist())
        assert len(s) == len(ws)
        for got, w in zip(s, ws):
            assert abs(Fraction(float(got)) - w) <= Fraction(1, 10 ** 9)
        off = oracle_offsets_of_flags(f)
        sc, _ = oracle.seg_sum_csr_bf16(xb, off)
        assert np.array_equal(sc, s)
    # values representable in both 16-bit formats: the two routes must agree exactly
    vals = rng.integers(-64, 65, 500).astype(np.float32) / 8
    f = (rng.random(500) < 0.1).astype(np.uint8)
    z16, a16 = oracle.seg_scan_f16(vals.astype(np.float16), f)
    zb, ab = oracle.seg_scan_bf16(gen.bf16_bits_of(vals), f)
    assert np.array_equal(z16, zb) and np.array_equal(a16, ab)


def oracle_offsets_of_flags(f):
    starts = [0] + [i for i in range(1, len(f)) if f[i]]
    return np.asarray(starts + [len(f)], np.int32)


# --------------------------------------------------------------------------
# COMPRESS (Section 2)
# --------------------------------------------------------------------------
def test_compress_of_the_worked_example_and_against_a_loop():
    g = load_golden("sec2_worked_example.txt")
    x, f = g["x"], g["f"]
    assert oracle.compress(np.asarray(x, np.int8), u8(f)).tolist() == g["compress_x_f"]
    assert oracle.compress(f16(x), u8(f)).tolist() == g["compress_x_f"]
    rng = np.random.default_rng(29)
    for trial in range(50):
        n = int(rng.integers(0, 200))
        f = (rng.random(n) < rng.choice([0.0, 0.1, 0.6, 1.0])).astype(np.uint8) * rng.integers(1, 256, n).astype(np.uint8)
        for x in (rng.integers(-128, 128, n).astype(np.int8), rng.standard_normal(n).astype(np.float16),
                  rng.integers(0, 65536, n).astype(np.uint16)):
            want = [x[i] for i in range(n) if f[i]]
            got = oracle.compress(x, f)
            assert got.dtype == x.dtype and got.tolist() == [v.item() for v in want]


# --------------------------------------------------------------------------
# segmented running maximum / minimum
# --------------------------------------------------------------------------
def test_segmented_running_max_and_min():
    g = load_golden("sec2_worked_example.txt")
    x, f = g["x"], g["f"]                       # x = (2,2,3,3,1,3,1,2), f = (1,0,1,0,0,1,0,0)
    assert oracle.seg_scan_minmax_i8(np.asarray(x, np.int8), u8(f)).tolist() == [2, 2, 3, 3, 3, 3, 3, 3]
    assert oracle.seg_scan_minmax_i8(np.asarray(x, np.int8), u8(f), want_min=True).tolist() == [2, 2, 3, 3, 1, 3, 1, 1]
    assert oracle.seg_scan_minmax_f16(f16(x), u8(f)).tolist() == [2, 2, 3, 3, 3, 3, 3, 3]
    rng = np.random.default_rng(37)
    for trial in range(60):
        n = int(rng.integers(1, 90))
        f = (rng.random(n) < rng.choice([0.0, 0.1, 0.5, 1.0])).astype(np.uint8)
        xi = rng.integers(-128, 128, n).astype(np.int8)
        xf = rng.standard_normal(n).astype(np.float16)
        for want_min in (False, True):
            pick = min if want_min else max
            def brute(v):
                out = []
                for i in range(n):
                    s = i
                    while s > 0 and not f[s]:
                        s -= 1
                    out.append(pick(v[s:i + 1]))
                return out
            assert oracle.seg_scan_minmax_i8(xi, f, want_min).tolist() == brute(xi.astype(int).tolist())
            assert oracle.seg_scan_minmax_f16(xf, f, want_min).tolist() == brute(xf.astype(np.float64).tolist())
        # duality, and the library routine when there is no flag
        assert np.array_equal(oracle.seg_scan_minmax_f16(xf, f, True), -oracle.seg_scan_minmax_f16(-xf, f, False))
        zero = np.zeros(n, np.uint8)
        assert np.array_equal(oracle.seg_scan_minmax_i8(xi, zero), np.maximum.accumulate(xi.astype(np.int32)))
        assert np.array_equal(oracle.seg_scan_minmax_f16(xf, zero, True), np.minimum.accumulate(xf.astype(np.float64)))


# --------------------------------------------------------------------------
# int8 values with an int64 result (no wrap)
# --------------------------------------------------------------------------
def test_wide_integer_scan():
    g = load_golden("sec2_worked_example.txt")
    x, f = g["x"], g["f"]                       # x = (2,2,3,3,1,3,1,2), f = (1,0,1,0,0,1,0,0)
    assert oracle.seg_scan_i8_wide(np.asarray(x, np.int8), u8(f)).tolist() == [2, 4, 3, 6, 7, 3, 4, 6]
    rng = np.random.default_rng(41)
    for trial in range(40):
        n = int(rng.integers(1, 200))
        xi = rng.integers(-128, 128, n).astype(np.int8)
        f = (rng.random(n) < rng.choice([0.0, 0.1, 0.5])).astype(np.uint8)
        want, run = [], 0
        for i in range(n):                      # the definition once more, on Python integers
            run = int(xi[i]) if (i == 0 or f[i]) else run + int(xi[i])
            want.append(run)
        assert oracle.seg_scan_i8_wide(xi, f).tolist() == want
        # its low 32 bits are the int32 scan; one segment is numpy's cumulative sum
        assert np.array_equal(oracle.seg_scan_i8_wide(xi, f).astype(np.int32), oracle.seg_scan_i8(xi, f))
        assert np.array_equal(oracle.seg_scan_i8_wide(xi, np.zeros(n, np.uint8)), np.cumsum(xi.astype(np.int64)))
    # past the int32 range: 2^25 values of -128 reach -2^32 (the int32 scan wraps to 0 there), closed form -128 (i + 1)
    n = 1 << 25
    z = oracle.seg_scan_i8_wide(np.full(n, -128, np.int8), np.zeros(n, np.uint8))
    idx = np.arange(0, n, 4097)
    assert z[-1] == -(1 << 32) and z[(1 << 24) + 5] == -128 * ((1 << 24) + 6) and np.array_equal(z[idx], -128 * (idx + 1))


def test_running_max_and_min_of_bfloat16_values():
    g = load_golden("sec2_worked_example.txt")
    x, f = g["x"], g["f"]                       # small integers: exact in bfloat16
    xb = gen.bf16_bits_of(np.asarray(x, np.float32))
    assert oracle.seg_scan_minmax_bf16(xb, u8(f)).tolist() == [2, 2, 3, 3, 3, 3, 3, 3]
    assert oracle.seg_scan_minmax_bf16(xb, u8(f), want_min=True).tolist() == [2, 2, 3, 3, 1, 3, 1, 1]
    rng = np.random.default_rng(43)
    for trial in range(40):
        n = int(rng.integers(1, 300))
        f = (rng.random(n) < rng.choice([0.0, 0.05, 0.5])).astype(np.uint8)
        # values that both 16-bit formats hold exactly: the fp16 function must agree
        small = rng.integers(-200, 200, n).astype(np.float32) / 4.0
        assert np.array_equal(oracle.seg_scan_minmax_bf16(gen.bf16_bits_of(small), f), oracle.seg_scan_minmax_f16(small.astype(np.float16), f))
        # the whole bfloat16 range, far beyond fp16's: brute force on the decoded values, duality, one segment = numpy
        xb = gen.bf16_bits_of((rng.standard_normal(n) * 10.0 ** rng.integers(-30, 30, n)).astype(np.float32))
        xd = oracle.bf16_to_double(xb)
        for want_min in (False, True):
            want, run = [], 0.0
            for i in range(n):
                run = xd[i] if (i == 0 or f[i]) else (min(run, xd[i]) if want_min else max(run, xd[i]))
                want.append(run)
            assert oracle.seg_scan_minmax_bf16(xb, f, want_min).tolist() == want
        assert np.array_equal(oracle.seg_scan_minmax_bf16(xb, f, True), -oracle.seg_scan_minmax_bf16(xb ^ np.uint16(0x8000), f, False))
        assert np.array_equal(oracle.seg_scan_minmax_bf16(xb, np.zeros(n, np.uint8)), np.maximum.accumulate(xd))


# ---------------------------------------------------------------------------
# the all-cores form of the fp16 scan (timed beside the one-core oracle by the benchmark)
# ---------------------------------------------------------------------------
def test_all_cores_scan_equals_the_sequential_oracle():
    # the paper's worked example of Section 2, cut into 3 chunks: (2,2,3 | 3,1,3 | 1,2) -> (2,4,3,6,7,3,4,6)
    x = np.array([2, 2, 3, 3, 1, 3, 1, 2], np.float16)
    f = np.array([1, 0, 1, 0, 0, 1, 0, 0], np.uint8)
    z, a, used = oracle.seg_scan_f16_all_cores(x, f, threads=3)
    assert used == 3 and z.tolist() == [2, 4, 3, 6, 7, 3, 4, 6] and a.tolist() == [2, 4, 3, 6, 7, 3, 4, 6]
    rng = np.random.default_rng(31)
    for n, p, threads in [(1, 0.5, 4), (7, 0.0, 8), (1000, 0.01, 7), (100003, 1e-4, 8), (100003, 0.0, 5), (4096, 1.0, 3),
                          (50000, 0.3, 1)]:
        x = rng.uniform(-1, 1, n).astype(np.float16)
        f = (rng.random(n) < p).astype(np.uint8)
        z0, a0 = oracle.seg_scan_f16(x, f)
        z1, a1, used = oracle.seg_scan_f16_all_cores(x, f, threads=threads)
        assert used == min(threads, n)
        # one more fp64 addition per element than the sequential recurrence: equal to ~1e-16 of the magnitudes
        assert np.all(np.abs(z1 - z0) <= 1e-13 * a0 + 1e-300), (n, p, threads)
        assert np.all(np.abs(a1 - a0) <= 1e-13 * a0 + 1e-300), (n, p, threads)
    # chunks without any start between chunks that have one: the carry passes through
    n = 90
    x = np.ones(n, np.float16)
    f = np.zeros(n, np.uint8)
    f[[5, 80]] = 1
    z, _, _ = oracle.seg_scan_f16_all_cores(x, f, threads=9)
    assert np.array_equal(z, oracle.seg_scan_f16(x, f)[0])


# ---------------------------------------------------------------------------
# element-wise integer product (Section 4.3.1, Lemma 4.4 / Corollary 4.5)
# ---------------------------------------------------------------------------
def test_mult_i8_against_python_integers_and_the_school_method():
    # every pair of int8 values against Python's integers
    v = np.arange(-128, 128, dtype=np.int64)
    xs, ys = np.repeat(v, 256), np.tile(v, 256)
    z = oracle.mult_i8(xs.astype(np.int8), ys.astype(np.int8))
    assert z.tolist() == [int(a) * int(b) for a, b in zip(xs.tolist(), ys.tolist())]
    # closed forms: x * 1 = x, x * 0 = 0, x * (-1) = -x, the two extremes
    x = v.astype(np.int8)
    assert np.array_equal(oracle.mult_i8(x, np.ones(256, np.int8)), v)
    assert not oracle.mult_i8(x, np.zeros(256, np.int8)).any()
    assert np.array_equal(oracle.mult_i8(x, np.full(256, -1, np.int8)), -v)
    assert oracle.mult_i8(np.array([-128, 127], np.int8), np.array([-128, 127], np.int8)).tolist() == [16384, 16129]
    # Lemma 4.4: the product is the sum of the partial terms of the school method, c_k = (bit k of y) ? x 2^k : 0,
    # with bit 7 of a two's-complement byte weighing -2^7 -- i.e. the last element of a segmented scan over the
    # terms of each product (Corollary 4.5), here with the oracle's own segmented sum over segments of 8 terms
    bits = (ys.astype(np.uint8)[:, None] >> np.arange(8)) & 1
    weights = np.array([1, 2, 4, 8, 16, 32, 64, -128], np.int64)
    terms = bits * xs[:, None] * weights[None, :]
    assert np.array_equal(terms.sum(axis=1), z)
    t16 = terms.astype(np.float16)                      # every term is exactly an fp16 value
    assert np.array_equal(t16.astype(np.int64), terms)
    off = (np.arange(xs.shape[0] + 1) * 8).astype(np.int32)
    sums, _ = oracle.seg_sum_csr_f16(t16.reshape(-1), off)
    assert np.array_equal(sums.astype(np.int64), z)
