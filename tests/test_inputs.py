"""The seeded input generators: determinism, chunk addressability, shapes."""
import numpy as np

import mmv_inputs as gen


def test_chunks_regenerate_independently(monkeypatch):
    monkeypatch.setattr(gen, "CHUNK", 1000)
    x = gen.f16_uniform(5, 3500)
    assert x.dtype == np.float16 and x.shape == (3500,)
    assert np.array_equal(x[2000:3000], gen.f16_uniform_chunk(5, 2, 1000))
    assert np.array_equal(x[3000:], gen.f16_uniform_chunk(5, 3, 500))
    assert np.array_equal(x, gen.f16_uniform(5, 3500))
    assert np.abs(x.astype(np.float32)).max() <= 1.0
    f = gen.flags(5, 3500, p=0.5)
    assert f[0] == 1 and f.dtype == np.uint8 and set(np.unique(f)) <= {0, 1}
    assert np.array_equal(f[1000:2000], gen.flags_chunk(5, 1, 1000, p=0.5))
    c = gen.flags(5, 3500, pattern="cycle123")
    assert c[:12].tolist() == [1, 1, 0, 1, 0, 0] * 2
    assert np.array_equal(c, np.tile(np.array([1, 1, 0, 1, 0, 0], np.uint8), 600)[:3500])
    z = gen.flags(5, 3500, p=0.0)
    assert z[0] == 1 and z[1:].sum() == 0
    assert gen.flags(5, 10, pattern="all").tolist() == [1] * 10


def test_config_shapes():
    x, f = gen.config1(1 << 12)
    assert x.shape == f.shape == (4096,) and 20 < f.sum() < 130
    x, off = gen.config2(1 << 16, max_len=512)
    assert off[0] == 0 and off[-1] == 1 << 16 and (np.diff(off) >= 1).all() and np.diff(off).max() <= 512
    x, f = gen.config3(1 << 14)
    assert x.dtype == np.int8 and x.min() >= -8 and x.max() <= 7
    rowptr, col, val, xv = gen.config4(rows=4096)
    lens = np.diff(rowptr)
    assert lens.min() >= 1 and lens.max() <= 10_000 and 0.3 < (lens == 1).mean() < 0.45
    assert col.shape[0] == val.shape[0] == rowptr[-1] and col.max() < 4096 and xv.dtype == np.float32
    rowptr, *_ = gen.config4(rows=4096, empty_fraction=0.1)
    assert 0.05 < (np.diff(rowptr) == 0).mean() < 0.15


def test_start_flags_of_offsets_agree_with_the_oracle_encoding():
    import oracle
    off = np.asarray([0, 0, 3, 3, 7, 12, 12], np.int32)
    f = gen.start_flags_of_offsets(off, 12)
    assert f.tolist() == [1, 0, 0, 1, 0, 0, 0, 1, 0, 0, 0, 0]
    assert np.array_equal(f, oracle.flags_from_offsets(off, 12))


def test_block_sparse_attention_pattern():
    # structure of the blocked sparse-attention matrices (Section 5: global, window and random blocks)
    b, r, dim = 4, 2, 512
    rowptr, col, val, x = gen.block_sparse_attention_csr(b, r, dim=dim)
    nb = dim // b
    lens = np.diff(rowptr.astype(np.int64))
    assert rowptr[0] == 0 and rowptr[-1] == col.shape[0] == val.shape[0] and x.shape == (dim,)
    assert (lens[:2 * b] == dim).all()                                   # two dense block rows
    assert (lens % b == 0).all() and lens[2 * b:].min() >= 4 * b and lens[2 * b:].max() <= (2 + 3 + r) * b
    dense = np.zeros((dim, dim), bool)
    for i in range(dim):
        c = col[rowptr[i]:rowptr[i + 1]]
        assert (np.diff(c) > 0).all() and c.min() >= 0 and c.max() < dim
        dense[i, c] = True
    blocks = dense.reshape(nb, b, nb, b)
    assert (blocks.all(axis=(1, 3)) | ~blocks.any(axis=(1, 3))).all()    # whole blocks only
    pat = blocks.any(axis=(1, 3))
    assert pat[:, :2].all() and pat[:2, :].all()                         # global block columns / rows
    idx = np.arange(nb)
    assert pat[idx, idx].all() and pat[idx[1:], idx[1:] - 1].all() and pat[idx[:-1], idx[:-1] + 1].all()     # window
    extra = pat[2:].sum(axis=1) - (pat[2:, :2].sum(axis=1))
    assert extra.max() <= 3 + r
    again = gen.block_sparse_attention_csr(b, r, dim=dim)
    assert all(np.array_equal(u, v) for u, v in zip((rowptr, col, val, x), again))


def test_row_length_mixes_have_the_table_shape():
    want = {"const2k": (2000, 2000, 2000), "mid": (18, 119, 204), "short": (1, 6, 44), "heavy": (1, 6, 395_000)}
    for kind in gen.ROW_LENGTH_MIXES:
        lens = gen.row_length_mix(kind, 700_000)
        lo, avg, hi = want[kind]
        assert lens.min() == lo and lens.max() == hi and abs(lens.mean() - avg) < 0.08 * avg + 0.3
    x, off = gen.seg_sum_row_mix("short", 1 << 16)
    assert off[0] == 0 and off[-1] == x.shape[0] and abs(x.shape[0] - (1 << 16)) < 3000
