"""GPU parity with the record store in a file (Section 3.5: sorted IDs, coalesced ranges,
io_uring reads with O_DIRECT into pinned staging, then copy and scatter): same lists, tables,
resident bytes and chain output as the oracle working from the bytes in memory."""
import numpy as np
import pytest
import torch

from paper_2608_22643_b200 import binding as nb
from paper_2608_22643_b200 import synth
from tests.harness import Pair, rel_l2, u16

pytestmark = pytest.mark.gpu

TINY = synth.CONFIGS["tiny"]
SMALL = synth.CONFIGS["small"]


def _run_steps(p, cfg, B=1, n=None):
    n = cfg.n_tokens if n is None else n
    xs = synth.hidden_states(cfg, n, batch=B)
    L, M = cfg.n_layers, cfg.d_ffn
    out = torch.empty((B, cfg.d_model), dtype=torch.float32, device="cuda")
    logits = torch.empty((B, L, M), dtype=torch.float32, device="cuda")
    warned = set()
    for t in range(n):
        nb.np_predict(p.eng.ctx, xs[t].cuda(), B, logits, None, p.eng.stream)
        warned.add(nb.np_step(p.eng.ctx, xs[t].cuda(), B, out, p.eng.stream, p.eng.copy_stream))
        torch.cuda.synchronize()
        res = p.ora.step(u16(xs[t]), logits_f32=logits.cpu().numpy())
        p.check_delta_against(res["deltas"])
        assert rel_l2(out.cpu().numpy(), res["x_final"]) < 1e-5, t
    p.check_resident_bytes()
    return warned


@pytest.mark.parametrize("io_depth", [0, 4, -1])
@pytest.mark.parametrize("policy", [nb.NP_EVICT_EXACT, nb.NP_EVICT_LRU])
@pytest.mark.parametrize("cfg", [TINY, SMALL])
def test_steps_from_a_store_file(tmp_path, cfg, policy, io_depth):
    p = Pair(cfg, policy=policy, transfer_mode=nb.NP_XFER_FILE, store_dir=tmp_path, io_depth=io_depth)
    try:
        _run_steps(p, cfg, n=6)
    finally:
        p.close()


@pytest.mark.parametrize("direct", [True, False])
def test_small_staging_splits_a_layer_into_chunks(tmp_path, direct):
    """Staging of 16 rows in parts of 4: the cold start (k rows per layer) and the steady
    deltas go through many chunks; the result does not change."""
    cfg = SMALL
    p = Pair(cfg, transfer_mode=nb.NP_XFER_FILE, store_dir=tmp_path, staging_rows=16, direct=direct)
    try:
        warned = _run_steps(p, cfg, n=4)
        assert nb.NP_W_CHUNKED in warned
    finally:
        p.close()


@pytest.mark.parametrize("mode", [nb.NP_XFER_FILE, nb.NP_XFER_HOST_GATHER])
@pytest.mark.parametrize("policy", [nb.NP_EVICT_EXACT, nb.NP_EVICT_LRU])
def test_mapped_staging_needs_no_staging_copy(tmp_path, mode, policy):
    """NP_F_MAPPED_STAGING: the scatter kernel reads the pinned staging through its device
    mapping (the paper's coherent mapped path); same result, chunked or not."""
    cfg = SMALL
    for staging_rows in (None, 16):
        p = Pair(cfg, policy=policy, transfer_mode=mode, store_dir=tmp_path, staging_rows=staging_rows,
                 flags=nb.NP_F_CHECK_BOUNDS | nb.NP_F_MAPPED_STAGING)
        try:
            _run_steps(p, cfg, n=4)
        finally:
            p.close()


def test_dense_prefix_is_filled_from_the_file(tmp_path):
    cfg = SMALL
    p = Pair(cfg, transfer_mode=nb.NP_XFER_FILE, store_dir=tmp_path, dense_layers=2, staging_rows=64)
    try:
        _run_steps(p, cfg, n=4)
    finally:
        p.close()


def test_batch_from_a_store_file(tmp_path):
    cfg, B = SMALL, 4
    p = Pair(cfg, max_batch=B, C=cfg.d_ffn // 2, transfer_mode=nb.NP_XFER_FILE, store_dir=tmp_path)
    try:
        _run_steps(p, cfg, B=B, n=4)
    finally:
        p.close()


def test_a_short_file_is_refused(tmp_path):
    cfg = TINY
    w1, w2 = synth.predictor_weights(cfg, "cpu")
    path = tmp_path / "short.bin"
    np.zeros(1000, dtype=np.uint8).tofile(path)
    ncfg = nb.make_config(cfg.n_layers, cfg.d_model, cfg.d_ffn, cfg.d_pred, cfg.top_k, cfg.capacity,
                          transfer_mode=nb.NP_XFER_FILE)
    with pytest.raises(nb.NpError) as e:
        nb.Engine(ncfg, w1.cuda(), w2.cuda(), None, store_path=str(path))
    assert e.value.code == nb.NP_E_INVAL and "store file" in str(e.value)
