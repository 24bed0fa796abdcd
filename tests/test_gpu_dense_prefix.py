"""GPU parity of the dense/sparse split (Section 3.1): the first d layers dense and fully
resident, the rest sparse through the delta path, in one residual chain."""
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
# four layers, so that dense and sparse parts both span more than one layer
DENSE = synth.StackConfig("dense", 4, 512, 2048, 64, 44, 60, 5, 13, 0.9)


@pytest.mark.parametrize("mode", [nb.NP_XFER_HOST_GATHER, nb.NP_XFER_ZERO_COPY, nb.NP_XFER_MEMCPY_RUNS])
@pytest.mark.parametrize("cfg,d", [(TINY, 1), (TINY, 2), (SMALL, 1), (SMALL, 2), (DENSE, 1), (DENSE, 3)])
def test_trajectory_with_dense_prefix(cfg, d, mode):
    p = Pair(cfg, transfer_mode=mode, dense_layers=d)
    try:
        L, M, W, D = cfg.n_layers, cfg.d_ffn, cfg.d_ffn // 32, cfg.d_model
        xs = synth.hidden_states(cfg, 5)
        logits = torch.zeros((1, L, M), dtype=torch.float32, device="cuda")
        bitmap = torch.full((L, W), -1, dtype=torch.int32, device="cuda")
        out = torch.empty((1, D), dtype=torch.float32, device="cuda")
        for t in range(5):
            x = xs[t].cuda()
            nb.np_predict(p.eng.ctx, x, 1, logits, bitmap, p.eng.stream)
            nb.np_step(p.eng.ctx, x, 1, out, p.eng.stream, p.eng.copy_stream)
            torch.cuda.synchronize()
            z32 = logits.cpu().numpy()
            assert not z32[0, :d].any()                      # dense layers are not scored
            assert not bitmap.cpu().numpy()[:d].any()        # and select nothing
            z = O.predict(u16(p.w1_cpu), u16(p.w2_cpu), u16(xs[t]), L, M)
            if d < L:
                assert rel_l2(z32[0, d:], z[0, d:]) < 1e-5
            full = z.astype(np.float32)
            full[0, d:] = z32[0, d:]                         # selection on the GPU's own logits
            res = p.ora.step(u16(xs[t]), logits_f32=full)
            assert (bitmap.cpu().numpy().view(np.uint32) == res["pred"]).all()
            cnt = p.check_delta_against(res["deltas"])
            assert (cnt[:d, nb.NP_CNT_PRED] == 0).all() and (cnt[:d, nb.NP_CNT_RESIDENT] == 0).all()
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < 1e-5, t
            # the chain alone, on the state the step left behind
            out2 = torch.empty_like(out)
            nb.np_mlp_chain(p.eng.ctx, x, 1, out2, p.eng.stream)
            torch.cuda.synchronize()
            assert rel_l2(out2.cpu().numpy(), res["x_final"]) < 1e-5
        p.check_resident_bytes()
    finally:
        p.close()


# row widths of the larger configurations (two 16-byte column pieces per thread of the dense-layer
# kernel, uneven splits of the row over the warps), on few rows; the 8192-wide one also has a
# predictor wider than the direct-load kernel's registers hold
WIDE13 = synth.StackConfig("wide13", 2, 5120, 1024, 640, 10, 25, 3, 21, 0.9)
WIDE70 = synth.StackConfig("wide70", 2, 8192, 512, 2048, 10, 25, 3, 22, 0.9)
ODDW = synth.StackConfig("oddw", 3, 2064, 608, 72, 10, 25, 3, 23, 0.9)    # D / 8 = 258 pieces


@pytest.mark.parametrize("cfg,d", [(WIDE13, 1), (WIDE13, 2), (WIDE70, 1), (ODDW, 2), (ODDW, 3)])
def test_dense_layers_at_other_row_widths(cfg, d):
    p = Pair(cfg, transfer_mode=nb.NP_XFER_HOST_GATHER, dense_layers=d)
    try:
        L, M = cfg.n_layers, cfg.d_ffn
        xs = synth.hidden_states(cfg, 3)
        logits = torch.zeros((1, L, M), dtype=torch.float32, device="cuda")
        out = torch.empty((1, cfg.d_model), dtype=torch.float32, device="cuda")
        for t in range(3):
            x = xs[t].cuda()
            nb.np_predict(p.eng.ctx, x, 1, logits, None, p.eng.stream)
            nb.np_step(p.eng.ctx, x, 1, out, p.eng.stream, p.eng.copy_stream)
            torch.cuda.synchronize()
            z = O.predict(u16(p.w1_cpu), u16(p.w2_cpu), u16(xs[t]), L, M).astype(np.float32)
            z32 = logits.cpu().numpy()
            if d < L:
                assert rel_l2(z32[0, d:], z[0, d:]) < 1e-5
                z[0, d:] = z32[0, d:]
            res = p.ora.step(u16(xs[t]), logits_f32=z)
            p.check_delta_against(res["deltas"])
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < 1e-5, t
        p.check_resident_bytes()
        p.eng.counters()
    finally:
        p.close()


def test_all_layers_dense():
    cfg = TINY
    p = Pair(cfg, dense_layers=cfg.n_layers)
    try:
        xs = synth.hidden_states(cfg, 2)
        out = torch.empty((1, cfg.d_model), dtype=torch.float32, device="cuda")
        for t in range(2):
            nb.np_step(p.eng.ctx, xs[t].cuda(), 1, out, p.eng.stream, p.eng.copy_stream)
            torch.cuda.synchronize()
            res = p.ora.step(u16(xs[t]))
            assert res["installed_bytes"] == 0
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < 1e-5
    finally:
        p.close()


def test_caller_bitmaps_and_single_layer_calls_respect_the_dense_prefix():
    cfg = SMALL
    d = 1
    p = Pair(cfg, dense_layers=d)
    try:
        L, M, W = cfg.n_layers, cfg.d_ffn, cfg.d_ffn // 32
        words = synth.random_bitmaps(L, M, p.k, 3, 2, 0.7)       # names rows of the dense layer too
        for t in range(2):
            nb.np_delta(p.eng.ctx, words[t].cuda(), p.eng.stream)
            nb.np_install(p.eng.ctx, 0, L, p.eng.copy_stream)
            masked = words[t].numpy().view(np.uint32).copy()
            masked[:d] = 0
            p.check_delta_against(p.ora.res.delta(masked))
        x = torch.zeros((1, cfg.d_model), dtype=torch.float32, device="cuda")
        with pytest.raises(nb.NpError) as e:
            nb.np_sparse_mlp(p.eng.ctx, 0, x, 1, x.clone(), p.eng.stream)
        assert e.value.code == nb.NP_E_INVAL
        nb.np_sparse_mlp(p.eng.ctx, d, x, 1, x.clone(), p.eng.stream)    # a sparse layer is fine
        torch.cuda.synchronize()
    finally:
        p.close()


def test_configurations_that_exclude_a_dense_prefix():
    for kw in (dict(max_batch=2, flags=nb.NP_F_NO_TENSOR_CORES), dict(flags=nb.NP_F_LAYER_LAUNCHES),
               dict(flags=nb.NP_F_DIRECT_LOADS)):
        cfg = nb.make_config(2, 256, 1024, 64, 102, 205, dense_layers=1, **kw)
        with pytest.raises(nb.NpError) as e:
            nb.np_query_sizes(cfg)
        assert e.value.code == nb.NP_E_INVAL


def test_lru_policy_reset_and_centroid_head_with_dense_prefix():
    cfg = SMALL
    d, K = 1, 32
    p = Pair(cfg, policy=nb.NP_EVICT_LRU, dense_layers=d, transfer_mode=nb.NP_XFER_HOST_GATHER, C=cfg.d_ffn // 3)
    try:
        L, M, W, D = cfg.n_layers, cfg.d_ffn, cfg.d_ffn // 32, cfg.d_model
        xs = synth.hidden_states(cfg, 6)
        out = torch.empty((1, D), dtype=torch.float32, device="cuda")
        logits = torch.zeros((1, L, M), dtype=torch.float32, device="cuda")

        def run(t):
            nb.np_predict(p.eng.ctx, xs[t].cuda(), 1, logits, None, p.eng.stream)
            nb.np_step(p.eng.ctx, xs[t].cuda(), 1, out, p.eng.stream, p.eng.copy_stream)
            torch.cuda.synchronize()
            full = O.predict(u16(p.w1_cpu), u16(p.w2_cpu), u16(xs[t]), L, M).astype(np.float32)
            full[0, d:] = logits.cpu().numpy()[0, d:]
            res = p.ora.step(u16(xs[t]), logits_f32=full)
            p.check_delta_against(res["deltas"])
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < 1e-5, t

        for t in range(3):
            run(t)
        # reset empties the sparse layers' residency; the dense records stay where they are
        nb.np_reset(p.eng.ctx, p.eng.stream)
        p.ora.res.reset()
        for t in range(3, 6):
            run(t)
        p.check_resident_bytes()
        # the centroid head selects nothing in a dense layer either
        bank = synth.centroid_bank(cfg, K).cuda()
        z = torch.randn((1, L, 2, K), dtype=torch.float32, device="cuda")
        words = torch.full((L, W), -1, dtype=torch.int32, device="cuda")
        nb.np_centroid_select(p.eng.ctx, z, 1, K, bank, None, words, p.eng.stream)
        torch.cuda.synchronize()
        w = words.cpu().numpy()
        assert not w[:d].any() and w[d:].any()
    finally:
        p.close()


@pytest.mark.parametrize("cfg,d,B", [(SMALL, 1, 2), (SMALL, 2, 9), (DENSE, 2, 16), (DENSE, 4, 5)])
def test_batches_with_dense_prefix(cfg, d, B):
    """Several sequences: dense layers run through the tensor-core batch kernels on whole
    records, every layer is scored (the logits keep their [B][L][M] layout) and the dense
    layers' bitmap rows are cleared."""
    p = Pair(cfg, max_batch=B, dense_layers=d, transfer_mode=nb.NP_XFER_ZERO_COPY, C=cfg.d_ffn // 2)
    try:
        L, M, W, D = cfg.n_layers, cfg.d_ffn, cfg.d_ffn // 32, cfg.d_model
        xs = synth.hidden_states(cfg, 3, batch=B)
        logits = torch.zeros((B, L, M), dtype=torch.float32, device="cuda")
        bitmap = torch.full((L, W), -1, dtype=torch.int32, device="cuda")
        out = torch.empty((B, D), dtype=torch.float32, device="cuda")
        for t in range(3):
            x = xs[t].cuda()
            nb.np_predict(p.eng.ctx, x, B, logits, bitmap, p.eng.stream)
            nb.np_step(p.eng.ctx, x, B, out, p.eng.stream, p.eng.copy_stream)
            torch.cuda.synchronize()
            z32 = logits.cpu().numpy()
            assert rel_l2(z32, O.predict(u16(p.w1_cpu), u16(p.w2_cpu), u16(xs[t]), L, M)) < 1e-5
            res = p.ora.step(u16(xs[t]), logits_f32=z32)
            assert (bitmap.cpu().numpy().view(np.uint32) == res["pred"]).all() and not res["pred"][:d].any()
            p.check_delta_against(res["deltas"])
            got = out.cpu().numpy()
            for b in range(B):
                assert rel_l2(got[b], res["x_final"][b]) < 1e-5, (t, b)
        p.check_resident_bytes()
    finally:
        p.close()
