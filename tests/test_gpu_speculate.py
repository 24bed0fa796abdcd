"""Speculative prefetch behind a step (the deeper prefetch pipeline the paper names as future work,
Section 6) on the GPU against the oracle: lists, tables and installed bytes bit-exact, the chain's
output unchanged."""
import numpy as np
import pytest
import torch

from oracle import np_oracle as O
from paper_2608_22643_b200 import binding as nb
from paper_2608_22643_b200 import synth
from tests.harness import Pair, rel_l2, u16

pytestmark = pytest.mark.gpu

TINY = synth.CONFIGS["tiny"]
SMALL = synth.CONFIGS["small"]


def _check_spec(p, specs):
    for l, (ids, slots) in enumerate(specs):
        got_ids, got_slots = p.eng.speculative_lists(l)
        assert got_ids.shape == ids.shape and (got_ids == ids).all(), l
        assert (got_slots == slots).all(), l


def _check_tables(p):
    for l in range(p.cfg.n_layers):
        st = p.eng.export_state(l)
        resident = O.bitmap_to_bool(st["resident"], p.cfg.d_ffn)
        assert O.validity_errors(st["slot_map"], st["owner"], resident, p.C) == [], l
        assert (st["slot_map"] == p.ora.res.S[l]).all() and (st["owner"] == p.ora.res.owner[l]).all(), l
        assert (st["resident"] == O.bool_to_bitmap(p.ora.res.R[l])).all() and (st["stamp"] == p.ora.res.stamp[l]).all(), l


@pytest.mark.parametrize("policy", [nb.NP_EVICT_EXACT, nb.NP_EVICT_LRU])
@pytest.mark.parametrize("mode", [nb.NP_XFER_MEMCPY_RUNS, nb.NP_XFER_HOST_GATHER, nb.NP_XFER_ZERO_COPY])
@pytest.mark.parametrize("cfg,B,extra", [(TINY, 1, 30), (SMALL, 1, 64), (SMALL, 3, 40)])
def test_step_with_speculative_rows(policy, mode, cfg, B, extra):
    """np_step with spec_rows = s: the rows ranked k+1 .. k+s of the step's own logits are made resident
    and transferred behind the step; every list, table and resident byte matches the oracle each step,
    and the next step's incoming rows are the oracle's (fewer than without the prefetch)."""
    p = Pair(cfg, policy=policy, max_batch=B, transfer_mode=mode, spec_rows=extra)
    plain = O.Engine(cfg.n_layers, cfg.d_model, cfg.d_ffn, cfg.d_pred, p.k, p.C, policy,
                     u16(p.w1_cpu), u16(p.w2_cpu), p.store_u16)
    try:
        xs = synth.hidden_states(cfg, 6, batch=B)
        L, M = cfg.n_layers, cfg.d_ffn
        out = torch.empty((B, cfg.d_model), dtype=torch.float32, device="cuda")
        logits = torch.empty((B, L, M), dtype=torch.float32, device="cuda")
        saved = 0
        for t in range(6):
            nb.np_predict(p.eng.ctx, xs[t].cuda(), B, logits, None, p.eng.stream)
            nb.np_step(p.eng.ctx, xs[t].cuda(), B, out, p.eng.stream, p.eng.copy_stream)
            torch.cuda.synchronize()
            z32 = logits.cpu().numpy()
            # what np_delta left behind is read from its lists; the tables already hold the speculative rows
            res = p.ora.step(u16(xs[t]), logits_f32=z32, spec_extra=extra)
            ref = plain.step(u16(xs[t]), logits_f32=z32)
            cnt = p.eng.counters()
            for l, d in enumerate(res["deltas"]):
                got = p.eng.delta_lists(l, cnt[l])
                for f in ("delta_ids", "delta_slots", "evict_ids", "active_ids", "active_slots"):
                    assert (got[f] == getattr(d, f)).all() and got[f].shape == getattr(d, f).shape, (t, l, f)
                assert cnt[l][nb.NP_CNT_RESIDENT] == int(p.ora.res.R[l].sum())
                saved += ref["deltas"][l].delta_ids.size - d.delta_ids.size
            _check_spec(p, res["specs"])
            _check_tables(p)
            p.check_resident_bytes()
            got_x = out.cpu().numpy()
            for b in range(B):
                assert rel_l2(got_x[b], res["x_final"][b] if B > 1 else res["x_final"]) < 1e-5, (t, b)
            assert (res["x_final"] == ref["x_final"]).all()        # the prefetch changes no result
        if policy == nb.NP_EVICT_EXACT:
            assert saved > 0
    finally:
        p.close()


def test_speculate_with_caller_candidates_and_limits():
    """np_speculate on caller bitmaps after np_delta: budget 0, a budget above the free slots, candidates
    that are all resident, and two calls in a row; then the transfer and the next step's delta."""
    cfg = SMALL
    p = Pair(cfg, transfer_mode=nb.NP_XFER_HOST_GATHER)
    try:
        L, M, W = cfg.n_layers, cfg.d_ffn, cfg.d_ffn // 32
        words = synth.random_bitmaps(L, M, p.k, 91, 4, 0.6)
        xs = synth.hidden_states(cfg, 4)
        out = torch.empty((1, cfg.d_model), dtype=torch.float32, device="cuda")
        rng = np.random.default_rng(3)
        for t in range(4):
            w = words[t].numpy().view(np.uint32)
            nb.np_step_selected(p.eng.ctx, xs[t].cuda(), 1, words[t].cuda(), out, p.eng.stream, p.eng.copy_stream)
            res = p.ora.step(u16(xs[t]), pred_words=w)
            p.check_delta_against(res["deltas"])
            for budget in (0, 17, 10 ** 6 if t == 2 else 5):
                cand = O.bool_to_bitmap(rng.random((L, M)) < 0.3)
                nb.np_speculate(p.eng.ctx, torch.from_numpy(cand.view(np.int32)).cuda(), min(budget, p.C), p.eng.stream)
                specs = p.ora.res.speculate(cand, min(budget, p.C))
                for l, (ids, slots) in enumerate(specs):
                    O.install(p.ora.backing, p.ora.gate, p.ora.up, p.ora.downT, l, ids, slots)
                _check_spec(p, specs)
                nb.np_install_speculative(p.eng.ctx, p.eng.copy_stream)
                _check_tables(p)
            # all resident now: candidates = the resident set itself bring nothing
            nb.np_speculate(p.eng.ctx, torch.from_numpy(p.ora.res.resident_words().view(np.int32)).cuda(), 50, p.eng.stream)
            assert all(ids.size == 0 for ids, _ in p.ora.res.speculate(p.ora.res.resident_words(), 50))
            assert all(p.eng.speculative_lists(l)[0].size == 0 for l in range(L))
            nb.np_install_speculative(p.eng.ctx, p.eng.copy_stream)
            p.check_resident_bytes()
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < 1e-5
    finally:
        p.close()


def test_speculation_call_order_errors():
    p = Pair(TINY)
    try:
        z = torch.zeros((TINY.n_layers, TINY.d_ffn // 32), dtype=torch.int32, device="cuda")
        with pytest.raises(nb.NpError) as e:
            nb.np_speculate(p.eng.ctx, z, 4, p.eng.stream)          # no np_delta yet
        assert e.value.code == nb.NP_E_STATE
        nb.np_delta(p.eng.ctx, z, p.eng.stream)
        with pytest.raises(nb.NpError) as e:
            nb.np_install_speculative(p.eng.ctx, p.eng.copy_stream)  # no np_speculate since that delta
        assert e.value.code == nb.NP_E_STATE
        with pytest.raises(nb.NpError):
            nb.np_speculate(p.eng.ctx, z, -1, p.eng.stream)
        nb.np_speculate(p.eng.ctx, z, 4, p.eng.stream)
        nb.np_install_speculative(p.eng.ctx, p.eng.copy_stream)
        p.eng.counters()
    finally:
        p.close()
