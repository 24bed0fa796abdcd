"""Pins for the oracle's residency manager: Eq. 2-3 identities, slot-map
invariants, paper-fixed special cases and a set-based brute force."""
import numpy as np
import pytest

from oracle import np_oracle as O
from paper_2608_22643_b200 import synth


def _words(T, L, M, n_set, seed, persistence=0.8):
    return synth.random_bitmaps(L, M, n_set, seed, T, persistence).numpy().view(np.uint32)


def test_validity_checker_accepts_any_correct_assignment_and_names_what_is_wrong():
    M, C = 64, 8
    R = np.zeros(M, bool)
    rows = np.array([3, 17, 40, 63])
    R[rows] = True
    P = np.zeros(M, bool)
    P[[3, 40, 50]] = True
    for slots in ([0, 1, 2, 3], [7, 2, 5, 0]):                # canonical order or not: both valid
        S = np.full(M, -1)
        S[rows] = slots
        owner = np.full(C, -1)
        owner[slots] = rows
        assert O.validity_errors(S, owner, R, C, P, np.array([40, 3])) == []
    S = np.full(M, -1)
    S[rows] = [0, 1, 1, 3]                                     # two rows in one slot
    owner = np.full(C, -1)
    owner[[0, 1, 3]] = [3, 40, 63]
    assert any("share a slot" in e for e in O.validity_errors(S, owner, R, C))
    S[rows] = [0, 1, 2, 9]                                     # slot outside the buffer
    assert any("outside" in e for e in O.validity_errors(S, owner, R, C))
    S[rows] = [0, 1, 2, 3]
    owner = np.full(C, -1)
    owner[[0, 1, 2, 3]] = [3, 17, 40, 62]                      # owner names the wrong row
    assert any("inverse" in e for e in O.validity_errors(S, owner, R, C))
    owner[[0, 1, 2, 3, 6]] = [3, 17, 40, 63, 5]                # a free slot with an owner
    assert any("free slot" in e for e in O.validity_errors(S, owner, R, C))
    owner[6] = -1
    S[5] = 4                                                   # mapped but not resident
    assert any("not resident" in e for e in O.validity_errors(S, owner, R, C))
    S[5] = -1
    assert any("active rows" in e for e in O.validity_errors(S, owner, R, C, P, np.array([3])))


def _check_tables(res: O.Residency):
    """S and owner are mutually inverse; S[n] >= 0 exactly on resident rows."""
    for l in range(res.L):
        assert O.validity_errors(res.S[l], res.owner[l], res.R[l], res.C) == []
    for l in range(res.L):
        R, S, owner = res.R[l], res.S[l], res.owner[l]
        assert ((S >= 0) == R).all()
        slots = S[R]
        assert len(set(slots.tolist())) == slots.size           # injective
        assert ((slots >= 0) & (slots < res.C)).all()
        assert (owner[slots] == np.flatnonzero(R)).all()
        used = np.zeros(res.C, bool)
        used[slots] = True
        assert (owner[~used] == -1).all()


@pytest.mark.parametrize("policy", [O.EVICT_EXACT, O.EVICT_LRU])
def test_set_identities_and_invariants(policy):
    L, M, k, C, T = 2, 256, 26, 60, 24
    words = _words(T, L, M, k, 3)
    res = O.Residency(L, M, C, policy)
    for t in range(T):
        R_prev = res.R.copy()
        S_prev = res.S.copy()
        P = O.bitmap_to_bool(words[t], M)
        out = res.delta(words[t])
        _check_tables(res)
        for l in range(L):
            d = out[l]
            Pset, Rp = set(np.flatnonzero(P[l])), set(np.flatnonzero(R_prev[l]))
            Din = set(d.delta_ids.tolist())
            E = set(d.evict_ids.tolist())
            # Eq. 2: incoming = predicted \ resident; nothing overflows here
            assert Din == Pset - Rp and d.overflow_ids.size == 0
            assert d.n_kept + len(Din) == d.n_pred == len(Pset)
            assert Din.isdisjoint(Rp) and (Din | (Pset & Rp)) == Pset
            # Eq. 3: outgoing rows are resident-but-not-predicted
            assert E <= (Rp - Pset) and E.isdisjoint(Pset)
            Rn = set(np.flatnonzero(res.R[l]))
            assert Rn == (Rp - E) | Din
            if policy == O.EVICT_EXACT:
                assert E == Rp - Pset and Rn == Pset          # resident set = predicted set
            else:
                assert Pset <= Rn <= (Rp | Pset)
                assert len(Rn) == min(C, len(Rp | Pset))
            # kept rows keep their slot; lists are ascending; active list = P and R
            kept = sorted(Pset & Rp)
            assert (res.S[l][kept] == S_prev[l][kept]).all()
            assert (np.diff(d.delta_ids) > 0).all() and (np.diff(d.evict_ids) > 0).all()
            assert (np.diff(d.delta_slots) > 0).all()
            assert d.active_ids.tolist() == sorted(Pset)
            assert (d.active_slots == res.S[l][d.active_ids]).all()
            assert (res.S[l][d.delta_ids] == d.delta_slots).all()
            assert (res.stamp[l][P[l]] == t).all()


def test_cold_start_fetches_full_set_into_first_slots():
    # Section 3.4: the first token has no previous active set.
    L, M, k, C = 1, 128, 12, 30
    words = _words(1, L, M, k, 4)
    res = O.Residency(L, M, C, O.EVICT_EXACT)
    d = res.delta(words[0])[0]
    P = np.flatnonzero(O.bitmap_to_bool(words[0], M)[0])
    assert d.delta_ids.tolist() == P.tolist()
    assert d.delta_slots.tolist() == list(range(k))
    assert d.evict_ids.size == 0 and d.n_kept == 0


def test_fixed_size_sets_reuse_exactly_the_freed_slots():
    # Section 3.4: with the buffer exactly as large as the active set, incoming
    # rows match outgoing rows and only freed slots are written.
    L, M, k, T = 1, 256, 32, 12
    words = _words(T, L, M, k, 5)
    res = O.Residency(L, M, k, O.EVICT_EXACT)
    res.delta(words[0])
    for t in range(1, T):
        S_prev = res.S[0].copy()
        d = res.delta(words[t])[0]
        assert d.delta_ids.size == d.evict_ids.size
        assert sorted(S_prev[d.evict_ids].tolist()) == d.delta_slots.tolist()


def test_same_prediction_moves_nothing_and_disjoint_replaces_all():
    L, M, k = 1, 128, 16
    a = np.zeros((1, M), bool); a[0, :k] = True
    b = np.zeros((1, M), bool); b[0, 64:64 + k] = True
    res = O.Residency(L, M, k, O.EVICT_EXACT)
    res.delta(O.bool_to_bitmap(a))
    d = res.delta(O.bool_to_bitmap(a))[0]
    assert d.delta_ids.size == 0 and d.evict_ids.size == 0 and d.n_kept == k
    d = res.delta(O.bool_to_bitmap(b))[0]
    assert d.delta_ids.tolist() == list(range(64, 64 + k))
    assert d.evict_ids.tolist() == list(range(k))
    assert d.delta_slots.tolist() == list(range(k))


def test_policies_coincide_when_capacity_equals_set_size():
    L, M, k, T = 2, 256, 30, 16
    words = _words(T, L, M, k, 6, persistence=0.7)
    ra, rb = O.Residency(L, M, k, O.EVICT_EXACT), O.Residency(L, M, k, O.EVICT_LRU)
    for t in range(T):
        da, db = ra.delta(words[t]), rb.delta(words[t])
        for l in range(L):
            for f in ("delta_ids", "delta_slots", "evict_ids", "active_ids", "active_slots"):
                assert (getattr(da[l], f) == getattr(db[l], f)).all()
        assert (ra.S == rb.S).all() and (ra.owner == rb.owner).all() and (ra.R == rb.R).all()


def test_lru_evicts_least_recently_predicted_with_index_ties():
    L, M, C = 1, 64, 4
    def bm(ids):
        b = np.zeros((1, M), bool); b[0, ids] = True
        return O.bool_to_bitmap(b)
    res = O.Residency(L, M, C, O.EVICT_LRU)
    res.delta(bm([10, 20]))          # t=0
    res.delta(bm([30, 40]))          # t=1: buffer full: 10,20 (stamp 0), 30,40 (stamp 1)
    d = res.delta(bm([30, 50]))[0]   # t=2: need one slot: evict 10 (stamp 0, lower index than 20)
    assert d.evict_ids.tolist() == [10] and d.delta_ids.tolist() == [50] and d.delta_slots.tolist() == [0]
    d = res.delta(bm([20, 60, 61]))[0]   # t=3: free 0, need 2: candidates 30(2),40(1),50(2) -> 40 then 30
    assert d.evict_ids.tolist() == [30, 40]
    assert d.delta_ids.tolist() == [60, 61]
    assert sorted(np.flatnonzero(res.R[0]).tolist()) == [20, 50, 60, 61]


@pytest.mark.parametrize("policy", [O.EVICT_EXACT, O.EVICT_LRU])
def test_overflow_truncates_highest_ids(policy):
    L, M, C = 1, 64, 5
    b = np.zeros((1, M), bool); b[0, [1, 3, 5, 7, 9, 11, 13]] = True
    res = O.Residency(L, M, C, policy)
    d = res.delta(O.bool_to_bitmap(b))[0]
    assert d.delta_ids.tolist() == [1, 3, 5, 7, 9] and d.overflow_ids.tolist() == [11, 13]
    assert d.active_ids.tolist() == [1, 3, 5, 7, 9]
    _check_tables(res)
    # next step, a different oversize set: kept rows stay, everything else is replaced
    b2 = np.zeros((1, M), bool); b2[0, [1, 3, 20, 21, 22, 23, 24]] = True
    d = res.delta(O.bool_to_bitmap(b2))[0]
    assert d.evict_ids.tolist() == [5, 7, 9]
    assert d.delta_ids.tolist() == [20, 21, 22] and d.overflow_ids.tolist() == [23, 24]
    assert d.n_kept + d.delta_ids.size + d.overflow_ids.size == d.n_pred == 7
    _check_tables(res)


def test_brute_force_with_python_sets():
    """An order-free restatement with dicts and sets on tiny shapes (EXACT policy)."""
    L, M, k, C, T = 1, 96, 9, 20, 30
    words = _words(T, L, M, k, 8, persistence=0.6)
    res = O.Residency(L, M, C, O.EVICT_EXACT)
    slot_of = {}
    for t in range(T):
        P = set(np.flatnonzero(O.bitmap_to_bool(words[t], M)[0]).tolist())
        d = res.delta(words[t])[0]
        for n in [n for n in slot_of if n not in P]:
            del slot_of[n]
        free = sorted(set(range(C)) - set(slot_of.values()))
        for n in sorted(P - set(slot_of)):
            slot_of[n] = free.pop(0)
        assert {int(n): int(res.S[0][n]) for n in np.flatnonzero(res.R[0])} == slot_of
        assert dict(zip(d.active_ids.tolist(), d.active_slots.tolist())) == slot_of
