"""Seeded synthetic inputs for the segmented scan / sum / SpMV workloads.

This module only draws random numbers and lays them out; it holds none of the
method's arithmetic and is the one piece of code that both the GPU tests and
the CPU oracle's tests may share.  Every array is produced in chunks of
``CHUNK`` elements, each from its own ``SeedSequence([BASE_SEED, config,
stream, chunk])``, so any chunk of a 2^30-element input can be regenerated
alone when results are compared piece by piece.

The workloads stand in for the paper's own inputs (segment lengths taken from
the rows of sparse-matrix collections, and uniformly random segment densities,
Section 5), whose data files are not available here.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

BASE_SEED = 250623906
CHUNK = 1 << 24

# stream ids
S_VALUES, S_FLAGS, S_LENGTHS, S_COLS, S_XVEC = 0, 1, 2, 3, 4


def _rng(config: int, stream: int, chunk: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([BASE_SEED, config, stream, chunk])))


def _chunks(n: int):
    c = 0
    while c * CHUNK < n:
        yield c, min(CHUNK, n - c * CHUNK)
        c += 1


# --------------------------------------------------------------------------
# values
# --------------------------------------------------------------------------
def f16_uniform_chunk(config: int, chunk: int, m: int = CHUNK, stream: int = S_VALUES) -> np.ndarray:
    """fp16 values: float32 uniform in [-1, 1) rounded to nearest-even fp16."""
    u = _rng(config, stream, chunk).random(CHUNK, dtype=np.float32)[:m]
    return (u * np.float32(2.0) - np.float32(1.0)).astype(np.float16)


def f16_normal_chunk(config: int, chunk: int, m: int = CHUNK, stream: int = S_VALUES) -> np.ndarray:
    g = _rng(config, stream, chunk).standard_normal(CHUNK, dtype=np.float32)[:m]
    return g.astype(np.float16)


def i8_uniform_chunk(config: int, chunk: int, m: int = CHUNK, lo: int = -8, hi: int = 7) -> np.ndarray:
    return _rng(config, S_VALUES, chunk).integers(lo, hi + 1, size=CHUNK, dtype=np.int8)[:m]


def _full(fn, n: int, dtype, *a, first_chunk: int = 0, **k) -> np.ndarray:
    """All chunks of an array; chunks are independent, so large arrays are filled by a few threads
    (numpy releases the GIL in the generators and conversions; the values do not depend on it).
    first_chunk > 0 gives the n elements that start at chunk `first_chunk` of a longer array
    (a shard of it: the same values the whole array holds there)."""
    out = np.empty(n, dtype)

    def fill(cm):
        c, m = cm
        out[c * CHUNK:c * CHUNK + m] = fn(*a, chunk=first_chunk + c, m=m, **k)

    todo = list(_chunks(n))
    workers = min(len(todo), os.cpu_count() or 1, 16)
    if workers <= 1:
        for cm in todo:
            fill(cm)
    else:
        with ThreadPoolExecutor(max_workers=workers) as ex:
            list(ex.map(fill, todo))
    return out


def f16_uniform(config: int, n: int, stream: int = S_VALUES, first_chunk: int = 0) -> np.ndarray:
    return _full(f16_uniform_chunk, n, np.float16, config, stream=stream, first_chunk=first_chunk)


def f16_normal(config: int, n: int, stream: int = S_VALUES) -> np.ndarray:
    return _full(f16_normal_chunk, n, np.float16, config, stream=stream)


def bf16_bits_of(x32: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round to nearest even (a data-type conversion,
    like the rounding to fp16 above; numpy has no bfloat16 type)."""
    u = np.ascontiguousarray(x32, np.float32).view(np.uint32)
    return ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)


def bf16_normal(config: int, n: int, stream: int = S_VALUES) -> np.ndarray:
    """Standard normal values as bfloat16 bit patterns (uint16)."""
    return bf16_bits_of(f16_normal(config, n, stream).astype(np.float32) * np.float32(1.0009765625))


def i8_uniform(config: int, n: int, lo: int = -8, hi: int = 7) -> np.ndarray:
    return _full(i8_uniform_chunk, n, np.int8, config, lo=lo, hi=hi)


# --------------------------------------------------------------------------
# start flags
# --------------------------------------------------------------------------
def flags_chunk(config: int, chunk: int, m: int = CHUNK, p: float = 1.0 / 64, pattern: str = "bernoulli") -> np.ndarray:
    """uint8 start flags of one chunk.

    pattern: "bernoulli" (probability p per element), "all" (every element
    starts a segment) or "cycle123" (segment lengths 1,2,3,1,2,3,...).  The
    first flag of the whole array is always 1.
    """
    if pattern == "all":
        f = np.ones(m, np.uint8)
    elif pattern == "cycle123":
        base = (chunk * CHUNK) % 6
        pat = np.array([1, 1, 0, 1, 0, 0], np.uint8)
        f = np.tile(np.roll(pat, -base), m // 6 + 1)[:m].copy()      # pat[(i + base) % 6] for i < m
    elif pattern == "bernoulli":
        if p <= 0.0:
            f = np.zeros(m, np.uint8)
        else:
            u = _rng(config, S_FLAGS, chunk).random(CHUNK, dtype=np.float32)[:m]
            f = (u < np.float32(p)).astype(np.uint8)
    else:
        raise ValueError(pattern)
    if chunk == 0 and m > 0:
        f[0] = 1
    return f


def flags(config: int, n: int, p: float = 1.0 / 64, pattern: str = "bernoulli", first_chunk: int = 0) -> np.ndarray:
    return _full(flags_chunk, n, np.uint8, config, p=p, pattern=pattern, first_chunk=first_chunk)


# --------------------------------------------------------------------------
# CSR offsets
# --------------------------------------------------------------------------
def offsets_uniform_lengths(config: int, n: int, max_len: int = 4096) -> np.ndarray:
    """int32 offsets of segments with lengths uniform in {1..max_len} covering exactly n."""
    if n == 0:
        return np.zeros(1, np.int32)
    rng = _rng(config, S_LENGTHS, 0)
    parts, total = [], 0
    while total < n:
        want = max(16, int(2.2 * (n - total) / (max_len + 1)) + 16)
        l = rng.integers(1, max_len + 1, size=want, dtype=np.int64)
        parts.append(l)
        total += int(l.sum())
    lens = np.concatenate(parts)
    cs = np.cumsum(lens)
    k = int(np.searchsorted(cs, n, side="left"))       # first index with cs >= n
    cs = cs[:k + 1]
    cs[k] = n                                          # truncate the last length
    off = np.empty(k + 2, np.int64)
    off[0] = 0
    off[1:] = cs
    return off.astype(np.int32)


def zipf_row_lengths(config: int, rows: int, s: float = 1.5, cap: int = 10_000,
                     empty_fraction: float = 0.0) -> np.ndarray:
    """Row lengths with P(k) proportional to k^-s on {1..cap} (inverse-CDF table)."""
    k = np.arange(1, cap + 1, dtype=np.float64)
    w = k ** (-s)
    cdf = np.cumsum(w / w.sum())
    rng = _rng(config, S_LENGTHS, 0)
    u = rng.random(rows)
    lens = np.searchsorted(cdf, u, side="left").astype(np.int64) + 1
    lens = np.minimum(lens, cap)
    if empty_fraction > 0.0:
        e = rng.random(rows) < empty_fraction
        lens[e] = 0
    return lens


def offsets_from_lengths(lens: np.ndarray) -> np.ndarray:
    off = np.zeros(lens.shape[0] + 1, np.int64)
    np.cumsum(lens, out=off[1:])
    if off[-1] >= 2 ** 31:
        raise ValueError("too many elements for int32 offsets")
    return off.astype(np.int32)


def start_flags_of_offsets(off: np.ndarray, n: int) -> np.ndarray:
    """The same segments as start flags: byte i is 1 iff a non-empty segment starts at i."""
    off = np.asarray(off, np.int64)
    f = np.zeros(n, np.uint8)
    starts = off[:-1][off[1:] > off[:-1]]
    f[starts] = 1
    return f


def csr_matrix(config: int, rows: int, cols: int, s: float = 1.5, cap: int = 10_000,
               empty_fraction: float = 0.0):
    """(rowptr int32, col int32, val fp16, x fp32) of a random CSR matrix.

    Row lengths follow the truncated power law above; column indices are
    uniform (unsorted, duplicates allowed); values uniform in [-1, 1); the
    dense vector is standard normal.
    """
    lens = zipf_row_lengths(config, rows, s, cap, empty_fraction)
    rowptr = offsets_from_lengths(lens)
    nnz = int(rowptr[-1])
    col = np.empty(nnz, np.int32)
    for c, m in _chunks(nnz):
        col[c * CHUNK:c * CHUNK + m] = _rng(config, S_COLS, c).integers(0, cols, size=CHUNK, dtype=np.int32)[:m]
    val = f16_uniform(config, nnz)
    x = _rng(config, S_XVEC, 0).standard_normal(cols, dtype=np.float32)
    return rowptr, col, val, x


# --------------------------------------------------------------------------
# the paper's other SpMV / segmented-sum workloads, as synthetic stand-ins
# --------------------------------------------------------------------------
BSA_BLOCKS = (2, 4, 16, 64)          # block sizes of the blocked sparse-attention matrices (Section 5)
BSA_RANDOM = (2, 4, 8)               # numbers of random attention blocks per block row


def block_sparse_attention_csr(block: int, random_blocks: int, dim: int = 65536, global_blocks: int = 2,
                               window_blocks: int = 3, config: int = 6):
    """(rowptr int32, col int32, val fp16, x fp32) of a matrix with the blocked sparse-attention
    pattern ("b-<block>_r-<random_blocks>"): dim x dim in dense blocks of `block` x `block`; block
    row I holds the first `global_blocks` block columns, the `window_blocks` block columns centred
    on I (clipped at the edges) and `random_blocks` block columns drawn uniformly (blocks that
    coincide are kept once); the first `global_blocks` block rows are dense.  Column indices are
    sorted inside every row.  Values are uniform in [-1, 1), the vector standard normal."""
    if dim % block:
        raise ValueError("dim must be a multiple of the block size")
    nb = dim // block
    g = min(global_blocks, nb)
    half = window_blocks // 2
    rnd = _rng(config, S_LENGTHS, block * 16 + random_blocks).integers(0, nb, size=(nb, random_blocks))
    ar = np.arange(block, dtype=np.int64)
    lens = np.empty(dim, np.int64)
    col_parts = []
    # the dense block rows
    lens[:g * block] = dim
    col_parts.append(np.tile(np.arange(dim, dtype=np.int32), g * block))
    step = max(1, 4096 // block)                     # block rows per round: bounds the temporaries
    for i0 in range(g, nb, step):
        i1 = min(nb, i0 + step)
        rows_i = np.arange(i0, i1, dtype=np.int64)
        cand = [np.broadcast_to(np.arange(g, dtype=np.int64), (i1 - i0, g))]
        cand.append(rows_i[:, None] + np.arange(-half, window_blocks - half, dtype=np.int64)[None, :])
        cand.append(rnd[i0:i1])
        c = np.concatenate(cand, axis=1)
        c = np.where((c >= 0) & (c < nb), c, nb)     # out of range -> sentinel
        c.sort(axis=1)
        dup = np.zeros(c.shape, bool)
        dup[:, 1:] = c[:, 1:] == c[:, :-1]
        valid = (c < nb) & ~dup                      # [block rows, candidates], ascending block columns
        k = valid.sum(axis=1)
        lens[i0 * block:i1 * block] = np.repeat(k * block, block)
        full = c[:, None, :, None] * block + ar[None, None, None, :]           # [I, row in block, candidate, column in block]
        full = np.broadcast_to(full, (i1 - i0, block, c.shape[1], block))
        mask = np.broadcast_to(valid[:, None, :, None], full.shape)
        col_parts.append(full[mask].astype(np.int32))
    rowptr = offsets_from_lengths(lens)
    col = np.concatenate(col_parts)
    nnz = int(rowptr[-1])
    assert col.shape[0] == nnz
    val = f16_uniform(config, nnz)
    x = _rng(config, S_XVEC, 0).standard_normal(dim, dtype=np.float32)
    return rowptr, col, val, x


# Row-length mixes with the minimum / average / maximum of the sparse matrices whose rows the
# paper takes its segment lengths from (Table 5.1): constant 2K; 18 / 119 / 204; 1 / 6 / 44;
# 1 / 6 / 395K (a few huge rows among very short ones).
ROW_LENGTH_MIXES = ("const2k", "mid", "short", "heavy")


def row_length_mix(kind: str, rows: int, config: int = 7) -> np.ndarray:
    rng = _rng(config, S_LENGTHS, ROW_LENGTH_MIXES.index(kind))
    if kind == "const2k":
        return np.full(rows, 2000, np.int64)
    if kind == "mid":
        return 18 + np.rint(186.0 * rng.beta(1.63, 1.37, size=rows)).astype(np.int64)      # 18..204, mean 119
    lens = np.minimum(rng.geometric(1.0 / 6.0, size=rows), 44).astype(np.int64)          # 1..44, mean just under 6
    if kind == "heavy":
        lens = np.minimum(rng.geometric(1.0 / 5.4, size=rows), 44).astype(np.int64)
        giants = rng.choice(rows, size=rows // 683_000 + 1, replace=False)
        lens[giants] = 395_000
    return lens


def seg_sum_row_mix(kind: str, n_target: int, config: int = 7):
    """(x fp16 N(0,1), offsets int32) with about n_target elements in rows drawn from the mix."""
    mean = {"const2k": 2000.0, "mid": 119.0, "short": 5.9, "heavy": 6.0}[kind]
    rows = max(1, int(n_target / mean))
    off = offsets_from_lengths(row_length_mix(kind, rows, config))
    return f16_normal(config, int(off[-1])), off


# --------------------------------------------------------------------------
# the five benchmark configurations (sizes can be scaled down for tests)
# --------------------------------------------------------------------------
C5_CASES = (
    ("p0", dict(p=0.0, pattern="bernoulli")),
    ("p1e-6", dict(p=1e-6, pattern="bernoulli")),
    ("p1e-3", dict(p=1e-3, pattern="bernoulli")),
    ("p0.1", dict(p=0.1, pattern="bernoulli")),
    ("p0.5", dict(p=0.5, pattern="bernoulli")),
    ("all", dict(p=1.0, pattern="all")),
    ("cycle123", dict(p=0.5, pattern="cycle123")),
)


def config1(n: int = 1 << 20):
    """Segmented scan: fp16 uniform values, Bernoulli(1/64) flags."""
    return f16_uniform(1, n), flags(1, n, p=1.0 / 64)


def config2(n: int = 1 << 26, max_len: int = 4096):
    """Segmented sum: fp16 normal values, CSR offsets with lengths uniform in {1..max_len}."""
    return f16_normal(2, n), offsets_uniform_lengths(2, n, max_len)


def config3(n: int = 1 << 28):
    """Segmented scan: int8 values uniform in {-8..7}, Bernoulli(1e-3) flags."""
    return i8_uniform(3, n), flags(3, n, p=1e-3)


def config4(rows: int = 1 << 20, cols: int | None = None, empty_fraction: float = 0.0):
    """CSR SpMV: power-law row lengths capped at 10^4."""
    return csr_matrix(4, rows, rows if cols is None else cols, empty_fraction=empty_fraction)


def config5_values(n: int = 1 << 30, first_chunk: int = 0):
    return f16_uniform(5, n, first_chunk=first_chunk)


def config5_flags(n: int, case: str, first_chunk: int = 0):
    kw = dict(C5_CASES)[case]
    return flags(5, n, first_chunk=first_chunk, **kw)
