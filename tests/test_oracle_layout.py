"""Pins the oracle's layout arithmetic to the figures the paper prints."""
import os

import numpy as np

from oracle import np_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLD, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_resident_buffer_sizes_match_paper():
    # Section 4.3: 5500 rows -> 129 MiB, 9865 rows -> 231 MiB per layer.
    for rows, D, mib in _rows("resident_buffer_sizes.txt"):
        got = O.resident_buffer_bytes(int(rows), int(D)) / 2**20
        assert round(got) == int(mib), (rows, got)
    # a padded or headered record (e.g. 24.5 KiB) would miss the second figure
    assert O.record_bytes(4096) == 24576
    assert round(9865 * (24.5 * 1024) / 2**20) != 231


def test_active_budgets_match_paper():
    # Section 4.1: K_max / intermediate size gives the stated active percentages.
    for kmax, M, pct in _rows("active_budgets.txt"):
        assert round(100.0 * int(kmax) / int(M), 1) == float(pct)
        # and the percent -> rows rule reproduces the budget to within rounding of the percent
        back = O.count_from_percent(round(float(pct)), int(M))
        assert abs(back - int(kmax)) <= int(M) * 0.005 + 1


def test_percent_rule_on_workload_shapes():
    assert O.count_from_percent(10, 1024) == 102
    assert O.count_from_percent(20, 1024) == 205
    assert O.count_from_percent(10, 11008) == 1101
    assert O.count_from_percent(25, 11008) == 2752
    assert [O.count_from_percent(p, 13824) for p in (8, 15, 25, 40)] == [1106, 2074, 3456, 5530]
    assert O.count_from_percent(5, 28672) == 1434
    assert O.count_from_percent(20, 28672) == 5734


def test_record_addressing_is_layer_major_and_contiguous():
    # Section 3.5: consecutive neuron IDs of a layer are consecutive byte ranges.
    M, D = 64, 16
    rec = O.record_bytes(D)
    assert O.record_offset_bytes(0, 0, M, D) == 0
    assert O.record_offset_bytes(0, 5, M, D) - O.record_offset_bytes(0, 4, M, D) == rec
    assert O.record_offset_bytes(1, 0, M, D) == M * rec
    # the offset agrees with numpy's own addressing of an [L, M, 3, D] uint16 array
    a = np.zeros((3, M, 3, D), dtype=np.uint16)
    assert O.record_offset_bytes(2, 7, M, D) == 2 * a.strides[0] + 7 * a.strides[1]


def test_bitmap_roundtrip_and_bit_order():
    bits = np.zeros(64, dtype=bool)
    bits[[0, 5, 31, 32, 63]] = True
    w = O.bool_to_bitmap(bits)
    assert w.tolist() == [(1 << 0) | (1 << 5) | (1 << 31), (1 << 0) | (1 << 31)]
    assert (O.bitmap_to_bool(w, 64) == bits).all()


def test_bf16_widening_exact():
    # 1.0, -2.0, 0.5, smallest normal, a value with all 7 mantissa bits set
    u = np.array([0x3F80, 0xC000, 0x3F00, 0x0080, 0x3FFF], dtype=np.uint16)
    got = O.bf16_to_f64(u)
    assert got.tolist() == [1.0, -2.0, 0.5, 2.0**-126, 1.0 + 127 / 128]


def test_coalesce_runs():
    assert O.coalesce_runs(np.array([], dtype=np.int32)) == []
    assert O.coalesce_runs(np.array([3, 4, 5, 9, 11, 12])) == [(3, 3), (9, 1), (11, 2)]
