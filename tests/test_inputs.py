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
