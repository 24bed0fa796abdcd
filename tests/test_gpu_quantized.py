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
    for kw in (dict(dense_layers=1),):
        cfg = nb.make_config(2, 256, 1024, 64, 102, 205, record_format=nb.NP_REC_INT8, **kw)
        with pytest.raises(nb.NpError) as e:
            nb.np_query_sizes(cfg)
        assert e.value.code == nb.NP_E_INVAL
    cfg = nb.make_config(2, 264, 1024, 64, 102, 205, record_format=nb.NP_REC_INT8)   # D % 16 != 0
    with pytest.raises(nb.NpError):
        nb.np_query_sizes(cfg)
