"""Pins of the oracle's Section 3.3 predictor (projection blocks -> residual trunk -> centroid
heads): the paper's parameter table, library routines for the two non-linearities, a scalar
restatement on tiny sizes, and structural properties of the trunk and the heads."""
import os

import numpy as np
import pytest
import torch

from oracle import np_oracle as O
from paper_2608_22643_b200 import synth


def _f64(w):
    """The weight dict of synth.trunk_weights as fp64 numpy arrays."""
    def a(t):
        return t.detach().cpu().to(torch.float64).numpy()
    out = {"K": w["K"], "emb": a(w["emb"]), "heads": a(w["heads"])}
    out["proj"] = [tuple(a(t) for t in blk) for blk in w["proj"]]
    out["cproj"] = tuple(a(t) for t in w["cproj"])
    out["blocks"] = [tuple(a(t) for t in blk) for blk in w["blocks"]]
    return out


def test_parameter_counts_match_the_papers_cost_table():
    want = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "predictor_cost_table.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                want[k] = float(v)
    got = O.trunk_param_counts(512, (4096, 4096, 128, 1), 512, 2048, 4, 31)
    for k, v in want.items():
        assert abs(got[k] / 1e6 - v) / v < 0.012, (k, got[k], v)       # the table is printed to 0.1 M
    assert abs(got["total"] / 1e6 - want["total"]) < 0.15
    assert got["total"] == sum(got[k] for k in want if k != "total")
    # the trunk does not grow with the layer count, the heads do, nothing grows with the FFN width
    more = O.trunk_param_counts(512, (4096, 4096, 128, 1), 512, 2048, 4, 62)
    assert more["residual_trunk"] == got["residual_trunk"] and more["output_heads"] == 2 * got["output_heads"]


def test_layer_norm_and_silu_against_torch():
    rng = np.random.default_rng(0)
    v = rng.standard_normal((5, 96)) * 3 + 1.5
    g, b = rng.standard_normal(96), rng.standard_normal(96)
    want = torch.nn.functional.layer_norm(torch.from_numpy(v), (96,), torch.from_numpy(g), torch.from_numpy(b), eps=O.LN_EPS)
    assert np.allclose(O.layer_norm(v, g, b), want.numpy(), rtol=1e-12, atol=1e-12)
    assert np.allclose(O.silu(v), torch.nn.functional.silu(torch.from_numpy(v)).numpy(), rtol=1e-12, atol=1e-14)
    # shift invariance, and the hand value silu(0) = 0, silu(x) -> x for large x
    assert np.allclose(O.layer_norm(v + 7.0, g, b), O.layer_norm(v, g, b), atol=1e-9)
    assert O.silu(np.array([0.0]))[0] == 0.0 and abs(O.silu(np.array([40.0]))[0] - 40.0) < 1e-12


def _scalar_forward(w, feats, cid):
    """The same computation with explicit loops (tiny sizes only)."""
    import math

    def lin(W, b, x):
        return [sum(W[r][c] * x[c] for c in range(len(x))) + b[r] for r in range(len(W))]

    def ln_silu(v, g, be):
        n = len(v)
        mu = sum(v) / n
        var = sum((t - mu) ** 2 for t in v) / n
        out = []
        for i, t in enumerate(v):
            y = (t - mu) / math.sqrt(var + O.LN_EPS) * g[i] + be[i]
            out.append(y / (1.0 + math.exp(-y)))
        return out

    z = []
    for (W, b, g, be), f in zip(w["proj"], feats):
        z += ln_silu(lin(W, b, list(f)), g, be)
    W, b, g, be = w["cproj"]
    z += ln_silu(lin(W, b, list(w["emb"][cid])), g, be)
    for (W1, b1, g, be, W2, b2) in w["blocks"]:
        h = ln_silu(lin(W1, b1, z), g, be)
        up = lin(W2, b2, h)
        z = [a + c for a, c in zip(z, up)]
    return [sum(row[c] * z[c] for c in range(len(z))) for row in w["heads"]]


def test_forward_matches_a_scalar_restatement_on_tiny_sizes():
    T, dims, K0, E, nb, nh, K = 4, (8, 16, 8, 1), 5, 8, 2, 3, 6
    w = _f64(synth.trunk_weights(T, dims, K0, E, nb, nh, K, seed=3))
    feats, ids = synth.trunk_features(dims, 2, K0, seed=3)
    for t in range(2):
        f = [x[t].to(torch.float64).numpy() for x in feats]
        got = O.trunk_forward(w, f, int(ids[t]))
        want = np.array(_scalar_forward(w, f, int(ids[t]))).reshape(nh, 2, K)
        assert got.shape == (nh, 2, K) and np.allclose(got, want, rtol=1e-10, atol=1e-12)


def test_structure_of_trunk_and_heads():
    T, dims, K0, E, nb, nh, K = 8, (16, 16, 8, 1), 7, 16, 3, 2, 4
    w = _f64(synth.trunk_weights(T, dims, K0, E, nb, nh, K, seed=5))
    feats, ids = synth.trunk_features(dims, 1, K0, seed=5)
    f = [x[0].to(torch.float64).numpy() for x in feats]
    # heads that copy single coordinates of z read the trunk output, in (layer, gate|up, k) order
    w["heads"] = np.zeros_like(w["heads"])
    for r in range(nh * 2 * K):
        w["heads"][r, r] = 1.0
    z_full = O.trunk_forward(w, f, int(ids[0])).reshape(-1)
    # residual blocks whose second matrices and biases vanish leave z as the concatenation of stage 1
    w0 = dict(w)
    w0["blocks"] = [(W1, b1, g, be, np.zeros_like(W2), np.zeros_like(b2)) for (W1, b1, g, be, W2, b2) in w["blocks"]]
    z0 = O.trunk_forward(w0, f, int(ids[0])).reshape(-1)
    first = O.silu(O.layer_norm(w["proj"][0][0] @ f[0] + w["proj"][0][1], w["proj"][0][2], w["proj"][0][3]))
    assert np.allclose(z0[:T], first) and not np.allclose(z_full[:T], first)
    # another centroid ID changes only the centroid half of the concatenation
    other = (int(ids[0]) + 1) % K0
    z1 = O.trunk_forward(w0, f, other).reshape(-1)
    n = nh * 2 * K
    cut = min(n, 4 * T)
    assert np.allclose(z1[:cut], z0[:cut])
    if n > 4 * T:
        assert not np.allclose(z1[4 * T:], z0[4 * T:])
    # the scalar feature: zero-padded columns do not matter
    assert w["proj"][3][0].shape[1] == 8 and not w["proj"][3][0][:, 1:].any()
