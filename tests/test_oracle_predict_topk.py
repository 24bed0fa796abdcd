"""Pins for the oracle's predictor forward and top-k selection."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import np_oracle as O


def _bf16_bits(vals):
    """fp32 values that are exactly representable in bf16 -> their bit patterns."""
    a = np.asarray(vals, dtype=np.float32)
    b = a.view(np.uint32)
    assert ((b & 0xFFFF) == 0).all(), "value not bf16-exact"
    return (b >> 16).astype(np.uint16)


def _small_exact(rng, shape):
    """Random multiples of 1/8 in [-4, 4): exact in bf16."""
    return rng.integers(-32, 32, size=shape).astype(np.float32) / 8.0


def test_predict_exact_rational_brute_force():
    # every product and sum is done in exact rational arithmetic by scalar loops
    rng = np.random.default_rng(1)
    L, M, H, D, B = 2, 32, 5, 7, 3
    w1 = _small_exact(rng, (H, D))
    w2 = _small_exact(rng, (L * M, H))
    x = _small_exact(rng, (B, D))
    z = O.predict(_bf16_bits(w1), _bf16_bits(w2), _bf16_bits(x), L, M)
    assert z.shape == (B, L, M)
    for b in range(B):
        h = []
        for m in range(H):
            acc = sum(Fraction(float(w1[m, j])) * Fraction(float(x[b, j])) for j in range(D))
            h.append(acc if acc > 0 else Fraction(0))
        for l in range(L):
            for n in range(M):
                want = sum(Fraction(float(w2[l * M + n, m])) * h[m] for m in range(H))
                assert z[b, l, n] == float(want)
    # the brute force exercises the ReLU: some pre-activations are negative
    assert (x @ w1.T < 0).any() and (x @ w1.T > 0).any()


def test_predict_structured_closed_form():
    # W1 = rectangular identity, W2 row r = (r + 1) * one-hot(r mod H):
    # logits[l, n] = (l*M + n + 1) * max(0, x[(l*M + n) mod H]); catches a
    # transposed operand, a wrong layer stride and a dropped ReLU.
    L, M, H, D = 3, 32, 4, 6
    w1 = np.zeros((H, D), np.float32)
    w1[np.arange(H), np.arange(H)] = 1.0
    w2 = np.zeros((L * M, H), np.float32)
    r = np.arange(L * M)
    w2[r, r % H] = (r + 1).astype(np.float32)
    x = np.array([[1.5, -2.0, 0.25, -0.5, 100.0, -100.0]], np.float32)
    z = O.predict(_bf16_bits(w1), _bf16_bits(w2), _bf16_bits(x), L, M)
    want = ((r + 1) * np.maximum(0.0, x[0, r % H])).reshape(L, M)
    assert (z[0] == want).all()


def test_predict_hidden_not_rounded():
    # h = 1 + 2^-20 is not representable in bf16 or fp32-product-of-bf16 rounding
    # to bf16; the logit must still carry it exactly in fp64.
    w1 = np.array([[1.0, 2.0**-20]], np.float32)
    w2 = np.zeros((32, 1), np.float32)
    w2[:, 0] = 1.0
    x = np.array([[1.0, 1.0]], np.float32)
    z = O.predict(_bf16_bits(w1), _bf16_bits(w2), _bf16_bits(x), 1, 32)
    assert z[0, 0, 0] == 1.0 + 2.0**-20


def test_order_key_is_monotone_and_total():
    vals = np.array([-np.inf, -3.5, -1e-30, -0.0, 0.0, 1e-30, 2.0, np.inf], np.float32)
    key = O.fp32_order_key(vals).astype(np.int64)
    assert (np.diff(key) > 0).all()       # strictly increasing, so +0 ranks above -0


def _topk_brute(z, k):
    B, L, M = z.shape
    bits = np.zeros((L, M), bool)
    for b in range(B):
        for l in range(L):
            keys = O.fp32_order_key(z[b, l])
            order = sorted(range(M), key=lambda n: (-int(keys[n]), n))
            for n in order[:k]:
                bits[l, n] = True
    return bits


@pytest.mark.parametrize("B", [1, 3])
def test_topk_against_full_sort(B):
    rng = np.random.default_rng(2)
    L, M, k = 3, 96, 13
    z = rng.standard_normal((B, L, M)).astype(np.float32)
    z[:, :, ::7] = z[:, :, 3:4]            # plenty of exact ties
    got = O.bitmap_to_bool(O.topk_bitmap(z, k), M)
    assert (got == _topk_brute(z, k)).all()
    if B == 1:
        assert (got.sum(axis=1) == k).all()
    else:
        assert (got.sum(axis=1) >= k).all() and (got.sum(axis=1) <= B * k).all()


def test_topk_degenerate_cases():
    L, M = 2, 64
    z = np.zeros((1, L, M), np.float32)
    # all-equal logits: ties go to the lowest indices
    got = O.bitmap_to_bool(O.topk_bitmap(z, 10), M)
    assert (got[:, :10]).all() and not got[:, 10:].any()
    assert not O.bitmap_to_bool(O.topk_bitmap(z, 0), M).any()
    assert O.bitmap_to_bool(O.topk_bitmap(z, M), M).all()
    # -0 loses to +0
    z2 = np.full((1, 1, 32), -0.0, np.float32)
    z2[0, 0, [9, 20]] = 0.0
    got = O.bitmap_to_bool(O.topk_bitmap(z2, 3), 32)[0]
    assert set(np.flatnonzero(got)) == {0, 9, 20}
    # a strictly larger value at a high index beats ties at low indices
    z3 = np.zeros((1, 1, 32), np.float32)
    z3[0, 0, 31] = 1.0
    got = O.bitmap_to_bool(O.topk_bitmap(z3, 2), 32)[0]
    assert set(np.flatnonzero(got)) == {0, 31}
    # negatives order correctly (larger magnitude is smaller)
    z4 = -np.arange(1, 33, dtype=np.float32).reshape(1, 1, 32)
    got = O.bitmap_to_bool(O.topk_bitmap(z4, 4), 32)[0]
    assert set(np.flatnonzero(got)) == {0, 1, 2, 3}
