"""Pins for the oracle's dense/sparse split (Section 3.1: the first d layers stay dense and
resident, the rest run sparse through resident buffers) and the memory rule for d."""
import numpy as np
import torch

from oracle import np_oracle as O
from paper_2608_22643_b200 import synth


def _dense_stack_fp64(cfg, x_u16):
    """The whole stack as a dense pre-normalised residual chain in torch's own silu / matmul (fp64)."""
    x = torch.from_numpy(O.bf16_to_f64(x_u16))
    store = synth.backing_store(cfg).to(torch.float64)                   # [L, M, 3, D]
    for l in range(cfg.n_layers):
        xn = x / torch.sqrt((x * x).mean(dim=-1, keepdim=True) + 1e-6)
        Wg, Wu, WdT = store[l, :, 0], store[l, :, 1], store[l, :, 2]
        x = x + (torch.nn.functional.silu(xn @ Wg.T) * (xn @ Wu.T)) @ WdT
    return x.numpy()


def _u16(t):
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def _engine(cfg, d, k=None, C=None):
    w1, w2 = synth.predictor_weights(cfg)
    store = _u16(synth.backing_store(cfg))
    k = cfg.top_k if k is None else k
    C = cfg.capacity if C is None else C
    return O.Engine(cfg.n_layers, cfg.d_model, cfg.d_ffn, cfg.d_pred, k, C, O.EVICT_EXACT, _u16(w1), _u16(w2),
                    store, dense_layers=d), store


def test_all_layers_dense_is_the_dense_stack():
    cfg = synth.CONFIGS["tiny"]
    eng, store = _engine(cfg, cfg.n_layers)
    x = _u16(synth.hidden_states(cfg, 1)[0])
    out = eng.step(x)
    want = _dense_stack_fp64(cfg, x)
    assert np.linalg.norm(out["x_final"] - want) / np.linalg.norm(want) < 1e-13
    assert not out["pred"].any() and out["installed_bytes"] == 0
    assert all(d.delta_ids.size == 0 and d.active_ids.size == 0 for d in out["deltas"])


def test_dense_prefix_equals_sparse_layers_with_every_row_active():
    # a dense layer is a sparse layer whose whole row set is predicted and resident
    cfg = synth.CONFIGS["tiny"]
    L, M, W = cfg.n_layers, cfg.d_ffn, cfg.d_ffn // 32
    a, _ = _engine(cfg, 1, k=cfg.top_k, C=M)
    b, _ = _engine(cfg, 0, k=cfg.top_k, C=M)
    xs = synth.hidden_states(cfg, 3)
    for t in range(3):
        x = _u16(xs[t])
        ra = a.step(x)
        words = ra["pred"].copy()
        words[0] = 0xFFFFFFFF                      # layer 0: every row
        rb = b.step(x, pred_words=words)
        assert np.allclose(ra["x_final"], rb["x_final"], rtol=1e-11, atol=1e-12)
        assert (ra["pred"][1:] == rb["pred"][1:]).all() and not ra["pred"][0].any()
        for l in range(1, L):
            assert (ra["deltas"][l].delta_ids == rb["deltas"][l].delta_ids).all()
            assert (ra["deltas"][l].active_slots == rb["deltas"][l].active_slots).all()


def test_plan_is_the_largest_prefix_that_fits():
    L, M, D, C = 32, 11008, 4096, 2752
    rec = O.record_bytes(D)
    dense, sparse = M * rec, C * rec
    fixed = 3 * 2**30
    for budget in [0, fixed + 32 * sparse - 1, fixed + 32 * sparse, fixed + 32 * sparse + (dense - sparse) * 5 + 7,
                   fixed + 32 * dense - 1, fixed + 32 * dense, 10**13]:
        d = O.dense_prefix_plan(L, M, D, C, budget, fixed)
        fits = [x for x in range(L + 1) if x * dense + (L - x) * sparse + fixed <= budget]
        assert d == (max(fits) if fits else -1)
    assert O.dense_prefix_plan(L, M, D, C, fixed + 32 * sparse, fixed) == 0
    assert O.dense_prefix_plan(L, M, D, C, fixed + 32 * sparse + 5 * (dense - sparse), fixed) == 5
    assert O.dense_prefix_plan(L, M, D, C, fixed + 32 * dense, fixed) == 32
    # more budget never shortens the prefix; a larger resident capacity never lengthens it
    ds = [O.dense_prefix_plan(L, M, D, C, b, fixed) for b in range(fixed, fixed + 33 * dense, dense // 3)]
    assert ds == sorted(ds)
    assert O.dense_prefix_plan(L, M, D, 2 * C, fixed + 20 * dense, fixed) <= O.dense_prefix_plan(
        L, M, D, C, fixed + 20 * dense, fixed)
