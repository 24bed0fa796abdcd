"""Pins for the oracle's centroid selection head (Section 3.3 heads, Section 3.4 intersection)."""
import numpy as np

from oracle import np_oracle as O


def _random_case(rng, B, L, K, M, density=0.3):
    W = M // 32
    z = rng.standard_normal((B, L, 2, K)).astype(np.float32)
    bits = rng.random((L, 2, K, M)) < density
    bank = O.bool_to_bitmap(bits.reshape(-1, M)).reshape(L, 2, K, W)
    return z, bits, bank


def test_scalar_loop_brute_force():
    # neuron n of layer l is active iff for SOME sequence both chosen masks hold n;
    # the arg-max is found by a plain scan with Python float comparison
    rng = np.random.default_rng(3)
    B, L, K, M = 3, 4, 7, 64
    z, bits, bank = _random_case(rng, B, L, K, M)
    ids, words = O.centroid_select(z, bank)
    got = O.bitmap_to_bool(words, M)
    for l in range(L):
        want = [False] * M
        for b in range(B):
            pick = []
            for h in range(2):
                best = 0
                for c in range(1, K):
                    if float(z[b, l, h, c]) > float(z[b, l, h, best]):
                        best = c
                pick.append(best)
            assert list(ids[b, l]) == pick
            for n in range(M):
                if bits[l, 0, pick[0], n] and bits[l, 1, pick[1], n]:
                    want[n] = True
        assert list(got[l]) == want


def test_ties_take_lower_id_and_zero_signs_are_ordered():
    L, K, M = 1, 6, 32
    z = np.full((1, L, 2, K), -1.0, np.float32)
    z[0, 0, 0, [2, 4]] = 5.0            # two equal maxima -> centroid 2
    z[0, 0, 1, 1] = -0.0                # +0 ranks above -0 in the fp32 total order
    z[0, 0, 1, 3] = 0.0
    bank = np.zeros((L, 2, K, 1), np.uint32)
    bank[0, 0, :, 0] = 1 << np.arange(K)
    bank[0, 1, :, 0] = 0xFFFFFFFF
    ids, words = O.centroid_select(z, bank)
    assert ids.tolist() == [[[2, 3]]]
    assert words.tolist() == [[1 << 2]]


def test_one_hot_logits_and_identity_bank():
    # a one-hot logit row selects exactly that centroid; with the up bank all ones the
    # result is the gate mask itself, with disjoint gate/up masks it is empty
    rng = np.random.default_rng(5)
    L, K, M = 3, 5, 96
    _, bits, bank = _random_case(rng, 1, L, K, M, 0.4)
    z = np.zeros((1, L, 2, K), np.float32)
    g = rng.integers(0, K, L)
    u = rng.integers(0, K, L)
    z[0, np.arange(L), 0, g] = 1.0
    z[0, np.arange(L), 1, u] = 1.0
    full = bank.copy()
    full[:, 1] = 0xFFFFFFFF
    ids, words = O.centroid_select(z, full)
    assert (ids[0, :, 0] == g).all() and (ids[0, :, 1] == u).all()
    for l in range(L):
        assert (words[l] == bank[l, 0, g[l]]).all()
    disjoint = bank.copy()
    disjoint[:, 1] = ~bank[:, 0, :, :][:, :1]       # every up mask = complement of gate mask 0
    z0 = np.zeros((1, L, 2, K), np.float32)          # all ties -> centroid 0 on both heads
    _, words0 = O.centroid_select(z0, disjoint)
    assert not words0.any()


def test_set_bounds_and_batch_union():
    # |A| <= min(|gate mask|, |up mask|) per sequence; the batched result is the OR of the
    # per-sequence results; it feeds the delta step like any predicted bitmap
    rng = np.random.default_rng(7)
    B, L, K, M = 4, 3, 9, 128
    z, bits, bank = _random_case(rng, B, L, K, M, 0.25)
    ids, words = O.centroid_select(z, bank)
    acc = np.zeros_like(words)
    for b in range(B):
        ids_b, w_b = O.centroid_select(z[b:b + 1], bank)
        assert (ids_b[0] == ids[b]).all()
        n = O.bitmap_to_bool(w_b, M).sum(axis=1)
        for l in range(L):
            assert n[l] <= min(bits[l, 0, ids[b, l, 0]].sum(), bits[l, 1, ids[b, l, 1]].sum())
        acc |= w_b
    assert (acc == words).all()
    res = O.Residency(L, M, M // 2)
    out = res.delta(words)
    for l in range(L):
        pred = np.flatnonzero(O.bitmap_to_bool(words[l:l + 1], M)[0])
        got = np.sort(np.concatenate([out[l].delta_ids, out[l].overflow_ids]))
        assert (got == pred).all()
