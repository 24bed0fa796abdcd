"""GPU parity of the shared predictor of Section 3.3 (projection blocks -> residual trunk ->
centroid heads) against the oracle, alone and feeding the centroid selection."""
import numpy as np
import pytest
import torch

from oracle import np_oracle as O
from paper_2608_22643_b200 import binding as nb
from paper_2608_22643_b200 import synth
from tests.harness import rel_l2
from tests.test_oracle_trunk import _f64

pytestmark = pytest.mark.gpu


def _run(T, dims, K0, E, nb_blocks, nh, K, seed, tokens=3):
    w = synth.trunk_weights(T, dims, K0, E, nb_blocks, nh, K, seed, device="cuda")
    wf = _f64(w)
    feats, ids = synth.trunk_features(dims, tokens, K0, seed)
    desc, table = nb.trunk_pack(w, nh)
    ws = torch.empty(nb.np_trunk_workspace_floats(desc), dtype=torch.float32, device="cuda")
    logits = torch.full((nh, 2, K), 9.0, dtype=torch.float32, device="cuda")
    s = torch.cuda.Stream()
    worst = 0.0
    for t in range(tokens):
        f_dev = [f[t].cuda() for f in feats]
        cid = ids[t:t + 1].cuda()
        nb.np_trunk_forward(desc, table, f_dev, cid, ws, logits, s)
        s.synchronize()
        want = O.trunk_forward(wf, [f[t].to(torch.float64).numpy() for f in feats], int(ids[t]))
        got = logits.cpu().numpy()
        worst = max(worst, rel_l2(got, want))
        # the decision downstream: the arg-max centroid of every head (both sides on the GPU's logits
        # would be bit-exact; here the oracle's own logits must lead to the same IDs unless two
        # logits are closer than the arithmetic resolves)
        top2 = np.sort(want, axis=-1)[..., -2:]
        clear = (top2[..., 1] - top2[..., 0]) > 1e-4 * np.abs(top2[..., 1]).max()
        assert (got.argmax(-1)[clear] == want.argmax(-1)[clear]).all()
    return worst


@pytest.mark.parametrize("shape", [
    # T, feature dims, K0, E, blocks, heads, K
    (8, (8, 16, 8, 1), 5, 8, 2, 3, 6),
    (64, (256, 256, 128, 1), 16, 64, 4, 5, 40),
    (32, (72, 40, 24, 3), 7, 24, 1, 2, 33),          # dims that are not powers of two, one block
    (16, (4096, 4096, 128, 1), 9, 2048, 0, 2, 16),   # the paper's input widths, no trunk block
])
def test_forward_matches_oracle(shape):
    T, dims, K0, E, nblk, nh, K = shape
    assert _run(T, dims, K0, E, nblk, nh, K, seed=11) < 2e-5


def test_forward_at_the_papers_sizes():
    """T = 512, four blocks, K = 512, 31 sparse layers, the layer-0 feature widths of the paper's
    model: 207 M parameters (414 MB in bf16)."""
    assert _run(512, (4096, 4096, 128, 1), 512, 2048, 4, 31, 512, seed=12, tokens=2) < 2e-5


def test_heads_feed_the_centroid_selection():
    """Head logits [n_heads][2][K] are the layout np_centroid_select reads for one sequence."""
    cfg = synth.StackConfig("sel", 3, 64, 256, 16, 10, 25, 2, 51, 0.9)
    T, dims, K0, E, nblk, K = 16, (64, 64, 16, 1), 8, 16, 2, 12
    nh = cfg.n_layers
    w = synth.trunk_weights(T, dims, K0, E, nblk, nh, K, 13, device="cuda")
    feats, ids = synth.trunk_features(dims, 1, K0, 13)
    desc, table = nb.trunk_pack(w, nh)
    ws = torch.empty(nb.np_trunk_workspace_floats(desc), dtype=torch.float32, device="cuda")
    logits = torch.empty((1, nh, 2, K), dtype=torch.float32, device="cuda")
    from tests.harness import Pair
    p = Pair(cfg, with_oracle=False)
    try:
        nb.np_trunk_forward(desc, table, [f[0].cuda() for f in feats], ids[:1].cuda(), ws, logits, p.eng.stream)
        bank = synth.centroid_bank(cfg, K)
        words = torch.zeros((nh, cfg.d_ffn // 32), dtype=torch.int32, device="cuda")
        sel = torch.zeros((1, nh, 2), dtype=torch.int32, device="cuda")
        nb.np_centroid_select(p.eng.ctx, logits, 1, K, bank.cuda(), sel, words, p.eng.stream)
        torch.cuda.synchronize()
        want_ids, want_words = O.centroid_select(logits.cpu().numpy(), bank.numpy().view(np.uint32))
        assert (sel.cpu().numpy() == want_ids).all()
        assert (words.cpu().numpy().view(np.uint32) == want_words).all()
    finally:
        p.close()


def test_argument_errors():
    w = synth.trunk_weights(8, (8, 8, 8, 1), 4, 8, 1, 2, 4, 1, device="cuda")
    desc, table = nb.trunk_pack(w, 2)
    ws = torch.empty(nb.np_trunk_workspace_floats(desc), dtype=torch.float32, device="cuda")
    out = torch.empty((2, 2, 4), dtype=torch.float32, device="cuda")
    f = [torch.zeros(8, device="cuda") for _ in range(4)]
    cid = torch.zeros(1, dtype=torch.int32, device="cuda")
    for bad in ("T", "n_features", "E", "n_blocks", "K"):
        d2 = nb.np_trunk_desc.from_buffer_copy(desc)
        setattr(d2, bad, {"T": 12, "n_features": 3, "E": 4, "n_blocks": 17, "K": 0}[bad])
        with pytest.raises(nb.NpError) as e:
            nb.np_trunk_forward(d2, table, f, cid, ws, out, None)
        assert e.value.code == nb.NP_E_INVAL
    with pytest.raises(nb.NpError):
        nb.np_trunk_forward(desc, table, f, None, ws, out, None)
    assert nb.np_trunk_forward(desc, table, f, cid, ws, out, None) == nb.NP_OK
    torch.cuda.synchronize()
