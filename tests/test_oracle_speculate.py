"""Pins of the oracle's speculative residency (the deeper prefetch pipeline of the paper's future
work, Section 6): it is a cache-only change.  None of these needs a GPU."""
import numpy as np
import pytest

from oracle import np_oracle as O
from paper_2608_22643_b200 import synth


def _bitmap(M, ids):
    b = np.zeros(M, dtype=bool)
    b[list(ids)] = True
    return O.bool_to_bitmap(b[None, :])


def test_hand_worked_example():
    """M = 32, C = 6: after a delta that makes {3, 9, 20} resident in slots 0..2, candidates
    {1, 9, 5, 30, 31} with budget 2 bring in rows 1 and 5 (9 is resident; lowest index first)
    in slots 3 and 4; nothing else moves."""
    r = O.Residency(1, 32, 6, O.EVICT_EXACT)
    r.delta(_bitmap(32, [3, 9, 20]))
    (ids, slots), = r.speculate(_bitmap(32, [1, 9, 5, 30, 31]), 2)
    assert ids.tolist() == [1, 5] and slots.tolist() == [3, 4]
    assert np.flatnonzero(r.R[0]).tolist() == [1, 3, 5, 9, 20]
    assert r.owner[0].tolist() == [3, 9, 20, 1, 5, -1]
    assert r.stamp[0][[1, 5]].tolist() == [-1, -1]            # never predicted: first to leave under LRU
    # the next token predicts {1, 3, 7}: row 1 is already there, only 7 is incoming; Eq. 3 frees the rest
    d, = r.delta(_bitmap(32, [1, 3, 7]))
    assert d.delta_ids.tolist() == [7] and d.n_kept == 2
    assert d.evict_ids.tolist() == [5, 9, 20]
    assert np.flatnonzero(r.R[0]).tolist() == [1, 3, 7]


def test_budget_capacity_and_empty_cases():
    r = O.Residency(1, 64, 4, O.EVICT_LRU)
    r.delta(_bitmap(64, [0, 1, 2]))
    assert r.speculate(_bitmap(64, [10, 11, 12]), 0)[0][0].size == 0          # no budget
    (ids, slots), = r.speculate(_bitmap(64, [10, 11, 12]), 5)                 # one free slot only
    assert ids.tolist() == [10] and slots.tolist() == [3]
    assert r.speculate(_bitmap(64, [11, 12]), 5)[0][0].size == 0              # full: nothing is evicted for a guess
    assert r.speculate(_bitmap(64, []), 5)[0][0].size == 0
    assert O.validity_errors(r.S[0], r.owner[0], r.R[0], 4) == []


@pytest.mark.parametrize("policy", [O.EVICT_EXACT, O.EVICT_LRU])
def test_never_evicts_keeps_tables_valid_and_fills_lowest_free_slots(policy):
    rng = np.random.default_rng(5)
    L, M, C = 3, 256, 60
    r = O.Residency(L, M, C, policy)
    for t in range(12):
        P = np.zeros((L, M), dtype=bool)
        for l in range(L):
            P[l, rng.choice(M, size=25, replace=False)] = True
        r.delta(O.bool_to_bitmap(P))
        R0, S0, owner0, stamp0 = r.R.copy(), r.S.copy(), r.owner.copy(), r.stamp.copy()
        cand = rng.random((L, M)) < 0.2
        budget = int(rng.integers(0, 30))
        specs = r.speculate(O.bool_to_bitmap(cand), budget)
        for l, (ids, slots) in enumerate(specs):
            want = np.flatnonzero(cand[l] & ~R0[l])
            free = np.flatnonzero(owner0[l] == -1)
            n = min(budget, want.size, free.size)
            assert ids.tolist() == want[:n].tolist() and slots.tolist() == free[:n].tolist()
            assert (r.R[l] >= R0[l]).all()                                    # nothing left
            keep = R0[l]
            assert (r.S[l][keep] == S0[l][keep]).all()                        # resident rows keep their slot
            assert (r.stamp[l] == stamp0[l]).all()
            assert (P[l] <= r.R[l]).all() or policy == O.EVICT_EXACT and P[l].sum() > C
            assert O.validity_errors(r.S[l], r.owner[l], r.R[l], C) == []


def test_exact_policy_next_delta_shrinks_by_the_speculative_rows_that_are_predicted():
    """Two residencies over the same predictions, one with speculation: under Eq. 3 the
    incoming set without speculation is the disjoint union of the incoming set with it and the
    speculative rows that the next token predicts."""
    rng = np.random.default_rng(11)
    L, M, C = 2, 512, 128
    a, b = O.Residency(L, M, C, O.EVICT_EXACT), O.Residency(L, M, C, O.EVICT_EXACT)
    prev_spec = [np.zeros(0, np.int32)] * L
    for t in range(10):
        P = np.zeros((L, M), dtype=bool)
        for l in range(L):
            P[l, rng.choice(M, size=50, replace=False)] = True
        words = O.bool_to_bitmap(P)
        da, db = a.delta(words), b.delta(words)
        for l in range(L):
            used = set(prev_spec[l].tolist()) & set(np.flatnonzero(P[l]).tolist())
            assert set(da[l].delta_ids.tolist()) == set(db[l].delta_ids.tolist()) | used
            assert not set(db[l].delta_ids.tolist()) & used
            assert set(da[l].active_ids.tolist()) == set(db[l].active_ids.tolist())     # act = P and R either way
        cand = rng.random((L, M)) < 0.15
        prev_spec = [ids for ids, _ in b.speculate(O.bool_to_bitmap(cand), 40)]


@pytest.mark.parametrize("policy", [O.EVICT_EXACT, O.EVICT_LRU])
def test_chain_output_does_not_depend_on_speculation(policy):
    """The whole step on the tiny stack, with and without the speculative prefetch: the output of
    every layer is bit-identical (the active rows are the same rows, whatever slots hold them), the
    installed rows hold their records' bytes, and with it no step brings in more demand rows."""
    cfg = synth.CONFIGS["tiny"]
    u16 = lambda t: t.view(__import__("torch").int16).numpy().view(np.uint16)
    w1, w2 = synth.predictor_weights(cfg)
    store = u16(synth.backing_store(cfg))
    mk = lambda: O.Engine(cfg.n_layers, cfg.d_model, cfg.d_ffn, cfg.d_pred, cfg.top_k, cfg.capacity, policy,
                          u16(w1), u16(w2), store)
    plain, spec = mk(), mk()
    xs = synth.hidden_states(cfg, 6)
    fewer = 0
    for t in range(6):
        z = O.predict(u16(w1), u16(w2), u16(xs[t]), cfg.n_layers, cfg.d_ffn).astype(np.float32)
        ra = plain.step(u16(xs[t]), logits_f32=z)
        rb = spec.step(u16(xs[t]), logits_f32=z, spec_extra=40)
        assert (ra["x_final"] == rb["x_final"]).all()
        for l in range(cfg.n_layers):
            assert (ra["deltas"][l].active_ids == rb["deltas"][l].active_ids).all()
            if policy == O.EVICT_EXACT:     # (under LRU the two caches hold different rows, so no order is implied)
                assert rb["deltas"][l].delta_ids.size <= ra["deltas"][l].delta_ids.size
            fewer += ra["deltas"][l].delta_ids.size - rb["deltas"][l].delta_ids.size
            ids = np.flatnonzero(spec.res.R[l])
            slots = spec.res.S[l][ids]
            assert (spec.gate[l, slots] == store[l, ids, 0]).all() and (spec.downT[l, slots] == store[l, ids, 2]).all()
            sp_ids, sp_slots = rb["specs"][l]
            assert sp_ids.size <= 40 and not set(sp_ids.tolist()) & set(rb["deltas"][l].active_ids.tolist())
    if policy == O.EVICT_EXACT:
        assert fewer > 0                    # the next-best rows of one token are often the next token's rows
