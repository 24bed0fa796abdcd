"""Pins for the oracle's install and sparse SwiGLU MLP."""
import math

import numpy as np
import torch

from oracle import np_oracle as O
from paper_2608_22643_b200 import synth

CFG = synth.CONFIGS["tiny"]


def _store():
    return synth.backing_store(CFG).view(torch.int16).numpy().view(np.uint16)


def test_install_places_exact_bytes_and_ignores_run_grouping():
    st = _store()
    L, M, D, C = CFG.n_layers, CFG.d_ffn, CFG.d_model, 16
    g = np.zeros((L, C, D), np.uint16); u = g.copy(); dn = g.copy()
    ids = np.array([3, 4, 5, 100, 1023], np.int32)
    slots = np.array([7, 0, 15, 2, 9], np.int32)
    nbytes = O.install(st, g, u, dn, 1, ids, slots)
    assert nbytes == ids.size * O.record_bytes(D)
    for n, s in zip(ids, slots):
        assert (g[1, s] == st[1, n, 0]).all() and (u[1, s] == st[1, n, 1]).all() and (dn[1, s] == st[1, n, 2]).all()
    untouched = np.setdiff1d(np.arange(C), slots)
    assert not g[1, untouched].any() and not g[0].any()


def test_all_rows_active_equals_dense_swiglu():
    # every row resident and active (k = C = M): the sparse sum is the dense MLP,
    # here in torch's own silu/matmul (fp64)
    st = _store()
    L, M, D = CFG.n_layers, CFG.d_ffn, CFG.d_model
    g = np.zeros((L, M, D), np.uint16); u = g.copy(); dn = g.copy()
    perm = np.random.default_rng(0).permutation(M).astype(np.int32)     # arbitrary slot order
    O.install(st, g, u, dn, 1, np.arange(M, dtype=np.int32), perm)
    x = synth.hidden_states(CFG, 2, batch=1)[:, 0].to(torch.float64)     # [2, D]
    y = O.sparse_mlp(g, u, dn, 1, perm, x.numpy())
    rec = synth.backing_store(CFG)[1].to(torch.float64)                  # [M, 3, D]
    Wg, Wu, WdT = rec[:, 0], rec[:, 1], rec[:, 2]
    want = (torch.nn.functional.silu(x @ Wg.T) * (x @ Wu.T)) @ WdT
    err = np.linalg.norm(y - want.numpy()) / np.linalg.norm(want.numpy())
    assert err < 1e-13


def test_scalar_loop_and_known_silu_values():
    st = _store()
    L, M, D = CFG.n_layers, CFG.d_ffn, CFG.d_model
    ids = np.array([5, 77, 900], np.int32)
    x = np.random.default_rng(1).standard_normal((1, D))
    y = O.sparse_mlp_from_store(st, 0, ids, x)
    want = [0.0] * D
    for n in ids:
        gr, ur, dr = (O.bf16_to_f64(st[0, n, p]) for p in range(3))
        gv = sum(float(gr[j]) * float(x[0, j]) for j in range(D))
        uv = sum(float(ur[j]) * float(x[0, j]) for j in range(D))
        a = gv / (1.0 + math.exp(-gv)) * uv
        for j in range(D):
            want[j] += a * float(dr[j])
    assert np.allclose(y[0], want, rtol=1e-12, atol=1e-18)
    # closed forms: one neuron, gate row = c * e_0, up row = e_1, down row = e_2
    D2 = 8
    for c, silu in ((0.0, 0.0), (1.0, 1.0 / (1.0 + math.exp(-1.0))), (-1.0, -1.0 / (1.0 + math.e))):
        rec = np.zeros((1, 1, 3, D2), np.float32)
        rec[0, 0, 0, 0] = c; rec[0, 0, 1, 1] = 1.0; rec[0, 0, 2, 2] = 1.0
        bits = (rec.view(np.uint32) >> 16).astype(np.uint16)
        xx = np.zeros((1, D2)); xx[0, 0] = 1.0; xx[0, 1] = 3.0
        yy = O.sparse_mlp_from_store(bits, 0, np.array([0]), xx)
        want = np.zeros(D2); want[2] = silu * 3.0
        assert np.allclose(yy[0], want, rtol=1e-15, atol=0)


def test_linearity_over_disjoint_sets_and_buffer_vs_store():
    st = _store()
    D, C = CFG.d_model, 64
    L = CFG.n_layers
    g = np.zeros((L, C, D), np.uint16); u = g.copy(); dn = g.copy()
    ids = np.arange(10, 10 + 40, dtype=np.int32) * 7 % CFG.d_ffn
    ids = np.unique(ids).astype(np.int32)
    slots = np.random.default_rng(2).permutation(C)[:ids.size].astype(np.int32)
    O.install(st, g, u, dn, 0, ids, slots)
    x = np.random.default_rng(3).standard_normal((3, D))
    y_all = O.sparse_mlp(g, u, dn, 0, slots, x)
    h = ids.size // 2
    y_a = O.sparse_mlp(g, u, dn, 0, slots[:h], x)
    y_b = O.sparse_mlp(g, u, dn, 0, slots[h:], x)
    assert np.allclose(y_all, y_a + y_b, rtol=1e-12, atol=1e-18)
    # through slots and straight from the store agree
    assert np.allclose(y_all, O.sparse_mlp_from_store(st, 0, ids, x), rtol=1e-13, atol=1e-18)
    # empty active set
    assert not O.sparse_mlp(g, u, dn, 0, np.zeros(0, np.int32), x).any()


def test_rms_normalize_pins():
    x = np.array([[3.0, -4.0, 0.0, 0.0]])
    # mean square = 25/4, so the scale is 1/2.5 (up to the 1e-6 epsilon)
    assert np.allclose(O.rms_normalize(x), x / 2.5, rtol=1e-6, atol=0)
    r = np.random.default_rng(5).standard_normal((3, 64)) * 7.0
    n = O.rms_normalize(r)
    assert np.allclose(np.sqrt((n * n).mean(axis=1)), 1.0, rtol=1e-6)
    assert np.allclose(O.rms_normalize(5.0 * r), n, rtol=1e-6)          # scale invariant
    assert np.allclose(n * np.sqrt((r * r).mean(axis=1, keepdims=True) + 1e-6), r, rtol=1e-12)
    assert not O.rms_normalize(np.zeros((1, 8))).any()                   # epsilon keeps 0/0 away


def test_engine_trajectory_consistency():
    """Whole-step driver: buffers always hold the right bytes for every resident
    row, and the chain through slots equals the chain from the store."""
    cfg = CFG
    w1, w2 = synth.predictor_weights(cfg)
    as_u16 = lambda t: t.view(torch.int16).numpy().view(np.uint16)
    st = _store()
    xs = synth.hidden_states(cfg, 6)
    for policy in (O.EVICT_EXACT, O.EVICT_LRU):
        eng = O.Engine(cfg.n_layers, cfg.d_model, cfg.d_ffn, cfg.d_pred, cfg.top_k, cfg.capacity,
                       policy, as_u16(w1), as_u16(w2), st)
        overlaps = []
        prev = None
        for t in range(6):
            out = eng.step(as_u16(xs[t]))
            P = O.bitmap_to_bool(out["pred"], cfg.d_ffn)
            assert (P.sum(axis=1) == cfg.top_k).all()
            for l in range(cfg.n_layers):
                R = np.flatnonzero(eng.res.R[l]); S = eng.res.S[l][R]
                assert (eng.gate[l, S] == st[l, R, 0]).all()
                assert (eng.up[l, S] == st[l, R, 1]).all()
                assert (eng.downT[l, S] == st[l, R, 2]).all()
            x = O.bf16_to_f64(as_u16(xs[t]))
            for l, d in enumerate(out["deltas"]):
                x = x + O.sparse_mlp_from_store(st, l, d.active_ids, O.rms_normalize(x))
            assert np.allclose(x, out["x_final"], rtol=1e-12, atol=1e-15)
            if prev is not None:
                overlaps.append((P & prev).sum() / P.sum())
            prev = P
        assert 0.4 < np.mean(overlaps) < 0.95
