"""Stage 3b of the file path on the CPU (Section 3.5): sorted IDs, adjacent IDs coalesced into
ranges, reads through io_uring or blocking preads, into a caller's buffer.  No GPU involved."""
import os

import numpy as np
import pytest

from paper_2608_22643_b200 import binding as nb

REC = 1536                      # a record of the tiny shape: 3 * 256 * 2 bytes, a multiple of 512


def _store(tmp_path, n_records, seed=0, base=0):
    rng = np.random.default_rng(seed)
    data = rng.integers(0, 256, size=base + n_records * REC, dtype=np.uint8)
    path = tmp_path / "store.bin"
    data.tofile(path)
    return path, data


def _aligned(nbytes, align=4096):
    raw = np.zeros(nbytes + align, dtype=np.uint8)
    skip = (-raw.ctypes.data) % align
    return raw[skip:skip + nbytes]


def _runs(ids):
    return 0 if len(ids) == 0 else 1 + int((np.diff(ids) != 1).sum())


@pytest.mark.parametrize("depth", [0, 4, 256, -1])
@pytest.mark.parametrize("pattern", ["scattered", "runs", "all", "one", "none"])
def test_reads_match_the_file_and_adjacent_ids_coalesce(tmp_path, depth, pattern):
    n = 700
    path, data = _store(tmp_path, n)
    rng = np.random.default_rng(3)
    if pattern == "scattered":
        ids = np.sort(rng.choice(n, 90, replace=False))
    elif pattern == "runs":
        starts = np.sort(rng.choice(n // 20, 9, replace=False)) * 20
        ids = np.concatenate([np.arange(s, s + 1 + i) for i, s in enumerate(starts)])
    elif pattern == "all":
        ids = np.arange(n)
    elif pattern == "one":
        ids = np.array([n - 1])
    else:
        ids = np.zeros(0, dtype=np.int64)
    dst = _aligned(max(1, len(ids)) * REC)
    dst[:] = 0xEE
    fd = os.open(path, os.O_RDONLY)
    try:
        ranges, ring = nb.np_read_records(fd, 0, REC, ids, dst, depth)
    finally:
        os.close(fd)
    want = data.reshape(n, REC)[ids].reshape(-1)
    assert (dst[:len(ids) * REC] == want).all()
    assert ranges == _runs(ids)
    if depth < 0:
        assert not ring


def test_ranges_longer_than_one_read_and_a_base_offset(tmp_path):
    """3000 adjacent records are 4.6 MB, cut into reads of 1 MB; the store starts 4096 bytes in."""
    n, base = 3000, 4096
    path, data = _store(tmp_path, n, seed=5, base=base)
    ids = np.arange(n)
    dst = _aligned(n * REC)
    fd = os.open(path, os.O_RDONLY)
    try:
        ranges, _ = nb.np_read_records(fd, base, REC, ids, dst, 8)
    finally:
        os.close(fd)
    assert ranges == 1
    assert (dst == data[base:]).all()


def test_direct_io_when_the_file_system_allows(tmp_path):
    n = 256
    path, data = _store(tmp_path, n, seed=7)
    try:
        fd = os.open(path, os.O_RDONLY | os.O_DIRECT)
    except OSError:
        pytest.skip("no O_DIRECT on this file system")
    ids = np.sort(np.random.default_rng(1).choice(n, 64, replace=False))
    dst = _aligned(len(ids) * REC)
    try:
        nb.np_read_records(fd, 0, REC, ids, dst, 32)
    finally:
        os.close(fd)
    assert (dst == data.reshape(n, REC)[ids].reshape(-1)).all()


def test_errors(tmp_path):
    path, data = _store(tmp_path, 10)
    dst = _aligned(20 * REC)
    fd = os.open(path, os.O_RDONLY)
    try:
        for ids in ([3, 2], [1, 1], [-1, 4]):
            with pytest.raises(nb.NpError) as e:
                nb.np_read_records(fd, 0, REC, np.array(ids), dst, 4)
            assert e.value.code == nb.NP_E_INVAL
        with pytest.raises(nb.NpError) as e:                      # past the end of the file
            nb.np_read_records(fd, 0, REC, np.array([8, 9, 10, 11]), dst, 4)
        assert e.value.code == nb.NP_E_IO
        with pytest.raises(nb.NpError) as e:
            nb.np_read_records(fd, 0, REC, np.array([8, 9, 10, 11]), dst, -1)
        assert e.value.code == nb.NP_E_IO
        with pytest.raises(nb.NpError) as e:
            nb.np_read_records(fd, 0, REC, np.array([1]), dst, 5000)
        assert e.value.code == nb.NP_E_INVAL
    finally:
        os.close(fd)
    with pytest.raises(nb.NpError) as e:
        nb.np_read_records(-1, 0, REC, np.array([1]), dst, 4)
    assert e.value.code == nb.NP_E_INVAL
