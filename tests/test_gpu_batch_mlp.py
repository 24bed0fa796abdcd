"""GPU parity of the batched sparse MLP (Section 3.4 applied to several sequences): the
tensor-core kernels and the plain-core kernels against the oracle, per layer and as a chain."""
import numpy as np
import pytest
import torch

from oracle import np_oracle as O
from paper_2608_22643_b200 import binding as nb
from paper_2608_22643_b200 import synth
from tests.harness import Pair, rel_l2, u16

pytestmark = pytest.mark.gpu

SMALL = synth.CONFIGS["small"]
# many tiles per block (k = 900 rows), so ring slots are reused within a layer
DENSE = synth.StackConfig("dense", 4, 512, 2048, 64, 44, 60, 5, 13, 0.9)
# model width that splits into five slices of 64 columns
ODD = synth.StackConfig("odd", 2, 320, 1024, 32, 25, 50, 4, 17, 0.9)
# narrow rows, very many of them: a block's share exceeds its activation chunk and its slot cache
WIDE = synth.StackConfig("wide", 1, 128, 20480, 16, 100, 100, 2, 19, 0.9)

TC, ALU = 0, nb.NP_F_NO_TENSOR_CORES
TC5 = nb.NP_F_TCGEN05_BATCH   # up phase on tcgen05 where the shape allows it (row widths that are multiples of 256)


def _install_random_sets(p, words):
    cfg = p.cfg
    nb.np_delta(p.eng.ctx, words.cuda(), p.eng.stream)
    nb.np_install(p.eng.ctx, 0, cfg.n_layers, p.eng.copy_stream)
    deltas = p.ora.res.delta(words.numpy().view(np.uint32))
    for l, d in enumerate(deltas):
        O.install(p.store_u16, p.ora.gate, p.ora.up, p.ora.downT, l, d.delta_ids, d.delta_slots)
    return deltas


@pytest.mark.parametrize("flags", [TC, ALU, TC5])
@pytest.mark.parametrize("cfg,B,ring", [(SMALL, 2, 0), (SMALL, 3, 0), (SMALL, 8, 0), (SMALL, 9, 0), (SMALL, 16, 0),
                                        (DENSE, 4, 0), (DENSE, 16, 0), (DENSE, 16, 3), (DENSE, 7, 2), (ODD, 5, 0),
                                        (ODD, 12, 0)])
def test_single_layer_matches_oracle(cfg, B, ring, flags):
    p = Pair(cfg, max_batch=B, flags=flags | nb.NP_F_CHECK_BOUNDS, ring_stages=ring)
    try:
        words = synth.random_bitmaps(cfg.n_layers, cfg.d_ffn, p.k, 5, 2, 0.7)
        rng = np.random.default_rng(B)
        for t in range(2):
            deltas = _install_random_sets(p, words[t])
            x = rng.standard_normal((B, cfg.d_model)).astype(np.float32)
            x[B - 1] *= 30.0                                   # sequences of different scale
            xd = torch.from_numpy(x).cuda()
            y = torch.full((B, cfg.d_model), 7.0, dtype=torch.float32, device="cuda")
            for l, d in enumerate(deltas):
                nb.np_sparse_mlp(p.eng.ctx, l, xd, B, y, p.eng.stream)
                p.eng.stream.synchronize()
                want = O.sparse_mlp(p.ora.gate, p.ora.up, p.ora.downT, l, d.active_slots, x.astype(np.float64))
                got = y.cpu().numpy()
                for b in range(B):
                    assert rel_l2(got[b], want[b]) < 1e-5, (t, l, b)
        p.eng.counters()                                        # no bounds or wait error was recorded
    finally:
        p.close()


@pytest.mark.parametrize("flags", [TC, ALU, TC5])
@pytest.mark.parametrize("cfg,B", [(SMALL, 2), (SMALL, 11), (DENSE, 16), (ODD, 6)])
def test_chain_matches_oracle(cfg, B, flags):
    """The residual chain with the pre-MLP normalisation, several tokens in a row (the
    accumulators that alternate between layers are left clean for the next call)."""
    p = Pair(cfg, max_batch=B, flags=flags | nb.NP_F_CHECK_BOUNDS, C=cfg.d_ffn // 2 if B > 4 else None)
    try:
        xs = synth.hidden_states(cfg, 4, batch=B)
        out = torch.empty((B, cfg.d_model), dtype=torch.float32, device="cuda")
        logits = torch.empty((B, cfg.n_layers, cfg.d_ffn), dtype=torch.float32, device="cuda")
        for t in range(4):
            nb.np_predict(p.eng.ctx, xs[t].cuda(), B, logits, None, p.eng.stream)
            nb.np_step(p.eng.ctx, xs[t].cuda(), B, out, p.eng.stream, p.eng.copy_stream)
            torch.cuda.synchronize()
            res = p.ora.step(u16(xs[t]), logits_f32=logits.cpu().numpy())
            p.check_delta_against(res["deltas"])
            got = out.cpu().numpy()
            for b in range(B):
                assert rel_l2(got[b], res["x_final"][b]) < 1e-5, (t, b)
            # the chain alone, on the state the step left behind, gives the same vectors
            out2 = torch.empty_like(out)
            nb.np_mlp_chain(p.eng.ctx, xs[t].cuda(), B, out2, p.eng.stream)
            torch.cuda.synchronize()
            assert rel_l2(out2.cpu().numpy(), res["x_final"]) < 1e-5
    finally:
        p.close()


def test_kernel_choice_follows_the_flag():
    """The library names the kernels it launches for a batch: the tcgen05 up kernel only with its flag and only for
    row widths it covers."""
    for cfg, flags, want in [(DENSE, TC, "k_mlp_tc_up + k_mlp_tc_down"), (DENSE, TC5, "k_mlp_up5 + k_mlp_tc_down"),
                             (ODD, TC5, "k_mlp_tc_up + k_mlp_tc_down")]:
        p = Pair(cfg, max_batch=16, flags=flags)
        try:
            assert nb.np_mlp_kernel_name(p.eng.ctx, 16) == want, (cfg.name, flags)
        finally:
            p.close()


@pytest.mark.parametrize("B", [3, 16])
def test_many_rows_per_block(B):
    """Every row of a 20480-row layer active: a block's share spans several activation chunks
    and more rows than its slot cache holds."""
    cfg = WIDE
    M = cfg.d_ffn
    p = Pair(cfg, max_batch=B, k=M, C=M)
    try:
        words = torch.full((cfg.n_layers, M // 32), -1, dtype=torch.int32)
        deltas = _install_random_sets(p, words)
        x = np.random.default_rng(1).standard_normal((B, cfg.d_model)).astype(np.float32)
        y = torch.empty((B, cfg.d_model), dtype=torch.float32, device="cuda")
        nb.np_sparse_mlp(p.eng.ctx, 0, torch.from_numpy(x).cuda(), B, y, p.eng.stream)
        p.eng.stream.synchronize()
        want = O.sparse_mlp(p.ora.gate, p.ora.up, p.ora.downT, 0, deltas[0].active_slots, x.astype(np.float64))
        assert rel_l2(y.cpu().numpy(), want) < 1e-5
        p.eng.counters()
    finally:
        p.close()
