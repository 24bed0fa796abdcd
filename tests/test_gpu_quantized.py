"""GPU parity with 8-bit record stores: the install path dequantises rows on their way into
the resident buffers; everything downstream is unchanged."""
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


@pytest.mark.parametrize("policy", [nb.NP_EVICT_EXACT, nb.NP_EVICT_LRU])
@pytest.mark.parametrize("mode", [nb.NP_XFER_MEMCPY_RUNS, nb.NP_XFER_HOST_GATHER, nb.NP_XFER_ZERO_COPY])
@pytest.mark.parametrize("cfg,B", [(TINY, 1), (SMALL, 1), (SMALL, 4)])
def test_trajectory_on_8bit_records(cfg, B, mode, policy):
    p = Pair(cfg, policy=policy, transfer_mode=mode, max_batch=B, record_format=nb.NP_REC_INT8,
             C=cfg.capacity if B == 1 else cfg.d_ffn // 2)
    try:
        assert p.eng.sizes.record_bytes == 3 * cfg.d_model + 16
        L, M, D = cfg.n_layers, cfg.d_ffn, cfg.d_model
        xs = synth.hidden_states(cfg, 5, batch=B)
        logits = torch.empty((B, L, M), dtype=torch.float32, device="cuda")
        out = torch.empty((B, D), dtype=torch.float32, device="cuda")
        for t in range(5):
            x = xs[t].cuda()
            nb.np_predict(p.eng.ctx, x, B, logits, None, p.eng.stream)
            nb.np_step(p.eng.ctx, x, B, out, p.eng.stream, p.eng.copy_stream)
            torch.cuda.synchronize()
            res = p.ora.step(u16(xs[t]), logits_f32=logits.cpu().numpy())
            p.check_delta_against(res["deltas"])
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < 1e-5, t
        p.check_resident_bytes()          # every resident row is bit-for-bit the dequantised record
    finally:
        p.close()


def test_small_staging_chunks_8bit_records():
    cfg = SMALL
    p = Pair(cfg, transfer_mode=nb.NP_XFER_HOST_GATHER, staging_rows=14, record_format=nb.NP_REC_INT8)
    try:
        words = synth.random_bitmaps(cfg.n_layers, cfg.d_ffn, p.k, 7, 3, 0.5)
        for t in range(3):
            nb.np_delta(p.eng.ctx, words[t].cuda(), p.eng.stream)
            rc = nb.np_install(p.eng.ctx, 0, cfg.n_layers, p.eng.copy_stream)
            assert rc == nb.NP_W_CHUNKED
            p.check_delta_against(p.ora.res.delta(words[t].numpy().view(np.uint32)))
        p.check_resident_bytes()
    finally:
        p.close()


def test_configurations_8bit_records_exclude():
    cfg = nb.make_config(2, 264, 1024, 64, 102, 205, record_format=nb.NP_REC_INT8)   # D % 16 != 0
    with pytest.raises(nb.NpError) as e:
        nb.np_query_sizes(cfg)
    assert e.value.code == nb.NP_E_INVAL


@pytest.mark.parametrize("cfg,d,B", [(TINY, 1, 1), (SMALL, 2, 1), (SMALL, 1, 3)])
def test_8bit_records_with_dense_prefix(cfg, d, B):
    """Dense layers of an 8-bit store are dequantised once at start-up, with the install path's rounding."""
    p = Pair(cfg, max_batch=B, dense_layers=d, record_format=nb.NP_REC_INT8, transfer_mode=nb.NP_XFER_HOST_GATHER,
             C=cfg.capacity if B == 1 else cfg.d_ffn // 2)
    try:
        assert p.eng.sizes.dense_bytes == d * cfg.d_ffn * 3 * cfg.d_model * 2
        L, M, D = cfg.n_layers, cfg.d_ffn, cfg.d_model
        xs = synth.hidden_states(cfg, 4, batch=B)
        logits = torch.zeros((B, L, M), dtype=torch.float32, device="cuda")
        out = torch.empty((B, D), dtype=torch.float32, device="cuda")
        for t in range(4):
            x = xs[t].cuda()
            nb.np_predict(p.eng.ctx, x, B, logits, None, p.eng.stream)
            nb.np_step(p.eng.ctx, x, B, out, p.eng.stream, p.eng.copy_stream)
            torch.cuda.synchronize()
            full = O.predict(u16(p.w1_cpu), u16(p.w2_cpu), u16(xs[t]), L, M).astype(np.float32)
            z32 = logits.cpu().numpy()
            lo = d if B == 1 else 0                 # one sequence: dense layers are not scored at all
            full[:, lo:] = z32[:, lo:]
            res = p.ora.step(u16(xs[t]), logits_f32=full)
            p.check_delta_against(res["deltas"])
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < 1e-5, t
        p.check_resident_bytes()                    # includes the dense buffer, bit for bit
    finally:
        p.close()
