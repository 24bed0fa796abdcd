"""GPU parity of the centroid selection head (Section 3.3 heads, Section 3.4 intersection)
against the oracle, alone and feeding the delta / install / MLP path."""
import numpy as np
import pytest
import torch

from oracle import np_oracle as O
from paper_2608_22643_b200 import binding as nb
from paper_2608_22643_b200 import synth
from tests.harness import Pair, REL_L2_TOL, rel_l2, u16

pytestmark = pytest.mark.gpu

TINY = synth.CONFIGS["tiny"]
SMALL = synth.CONFIGS["small"]


def _select(p, logits, B, K, bank_dev):
    L, W = p.cfg.n_layers, p.cfg.d_ffn // 32
    ids = torch.full((B, L, 2), -7, dtype=torch.int32, device="cuda")
    words = torch.full((L, W), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    nb.np_centroid_select(p.eng.ctx, logits, B, K, bank_dev, ids, words, p.eng.stream)
    torch.cuda.synchronize()
    return ids.cpu().numpy(), words.cpu().numpy().view(np.uint32)


@pytest.mark.parametrize("cfg,B,K", [(TINY, 1, 5), (TINY, 3, 64), (SMALL, 1, 300), (SMALL, 4, 1000), (SMALL, 2, 1)])
def test_select_matches_oracle_bit_for_bit(cfg, B, K):
    p = Pair(cfg, max_batch=B, with_oracle=False)
    try:
        L = cfg.n_layers
        bank = synth.centroid_bank(cfg, K)
        rng = np.random.default_rng(cfg.seed + K)
        z = rng.standard_normal((B, L, 2, K)).astype(np.float32)
        # ties at the maximum, signed zeros and infinities in some rows
        if K >= 5:
            z[0, 0, 0, [1, 3]] = z[0, 0, 0].max() + 1.0
            z[-1, -1, 1, :] = -0.0
            z[-1, -1, 1, K // 2] = 0.0
            z[0, -1, 0, K - 1] = np.inf
            z[0, -1, 0, 0] = -np.inf
            z[0, 0, 1, :] = (rng.standard_normal(K) * 1e-42).astype(np.float32)    # a head whose logits are all denormal
        ids, words = _select(p, torch.from_numpy(z).cuda(), B, K, bank.cuda())
        want_ids, want_words = O.centroid_select(z, bank.numpy().view(np.uint32))
        assert (ids == want_ids).all()
        assert (words == want_words).all()
        # without the optional ID output the bitmap is the same
        W = cfg.d_ffn // 32
        words2 = torch.zeros((L, W), dtype=torch.int32, device="cuda")
        nb.np_centroid_select(p.eng.ctx, torch.from_numpy(z).cuda(), B, K, bank.cuda(), None, words2, p.eng.stream)
        torch.cuda.synchronize()
        assert (words2.cpu().numpy().view(np.uint32) == want_words).all()
    finally:
        p.close()


def test_argument_errors():
    p = Pair(TINY, max_batch=2, with_oracle=False)
    try:
        L, W, K = TINY.n_layers, TINY.d_ffn // 32, 8
        z = torch.zeros((2, L, 2, K), dtype=torch.float32, device="cuda")
        bank = synth.centroid_bank(TINY, K).cuda()
        words = torch.zeros((L, W), dtype=torch.int32, device="cuda")
        for args in [(None, 1, K, bank, None, words), (z, 1, K, None, None, words), (z, 1, K, bank, None, None),
                     (z, 3, K, bank, None, words), (z, 0, K, bank, None, words), (z, 1, 0, bank, None, words)]:
            with pytest.raises(nb.NpError) as e:
                nb.np_centroid_select(p.eng.ctx, *args, p.eng.stream)
            assert e.value.code == nb.NP_E_INVAL
    finally:
        p.close()


@pytest.mark.parametrize("policy", [nb.NP_EVICT_EXACT, nb.NP_EVICT_LRU])
@pytest.mark.parametrize("cfg,B,K", [(TINY, 1, 16), (SMALL, 3, 64)])
def test_centroid_heads_drive_the_whole_path(cfg, B, K, policy):
    """Head logits from the predictor kernels -> centroid selection -> delta -> install ->
    MLP chain, every stage through the C ABI; the selection is taken on the GPU's own logits
    on both sides, lists and tables are bit-exact, the chain output is within tolerance."""
    p = Pair(cfg, policy=policy, max_batch=B, transfer_mode=nb.NP_XFER_HOST_GATHER,
             C=cfg.capacity if B == 1 else cfg.d_ffn // 2)
    try:
        L, D, H, W = cfg.n_layers, cfg.d_model, cfg.d_pred, cfg.d_ffn // 32
        w2c = synth.centroid_head_weights(cfg, K)
        w2c_dev = w2c.cuda()
        bank = synth.centroid_bank(cfg, K)
        bank_dev = bank.cuda()
        bank_u32 = bank.numpy().view(np.uint32)
        xs = synth.hidden_states(cfg, cfg.n_tokens, batch=B)
        logits = torch.empty((B, L, 2, K), dtype=torch.float32, device="cuda")
        words = torch.empty((L, W), dtype=torch.int32, device="cuda")
        out = torch.empty((B, D), dtype=torch.float32, device="cuda")
        sizes = set()
        for t in range(cfg.n_tokens):
            x = xs[t].cuda()
            nb.np_predict_logits_noalloc(p.eng.w1, w2c_dev, x, B, L, D, 2 * K, H, logits, p.eng.stream)
            nb.np_centroid_select(p.eng.ctx, logits, B, K, bank_dev, None, words, p.eng.stream)
            nb.np_delta(p.eng.ctx, words, p.eng.stream)
            nb.np_install(p.eng.ctx, 0, L, p.eng.copy_stream)
            nb.np_mlp_chain(p.eng.ctx, x, B, out, p.eng.stream)
            torch.cuda.synchronize()
            z32 = logits.cpu().numpy()
            _, want_words = O.centroid_select(z32, bank_u32)
            assert (words.cpu().numpy().view(np.uint32) == want_words).all(), t
            res = p.ora.step(u16(xs[t]), pred_words=want_words)
            cnt = p.check_delta_against(res["deltas"])
            sizes.update(int(c[nb.NP_CNT_PRED]) for c in cnt)
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < REL_L2_TOL, t
            # the oracle's own head logits agree with the GPU's
            z = O.predict(u16(p.w1_cpu), u16(w2c), u16(xs[t]), L, 2 * K)
            assert rel_l2(z32.reshape(B, L, 2 * K), z) < 1e-5
        p.check_resident_bytes()
        assert len(sizes) > 1          # set sizes vary, unlike the fixed-k selection
    finally:
        p.close()


@pytest.mark.parametrize("dense", [0, 1])
def test_step_from_a_supplied_bitmap(dense):
    """np_step_selected = np_step with the predictor's result replaced by the caller's bitmap:
    same lists, tables, resident bytes and chain output as the oracle stepping on those sets."""
    cfg, B = SMALL, 1
    p = Pair(cfg, max_batch=B, dense_layers=dense)
    try:
        L, D, W = cfg.n_layers, cfg.d_model, cfg.d_ffn // 32
        xs = synth.hidden_states(cfg, cfg.n_tokens, batch=B)
        words = synth.random_bitmaps(L, cfg.d_ffn, p.k, 9, cfg.n_tokens, 0.8)
        out = torch.empty((B, D), dtype=torch.float32, device="cuda")
        for t in range(cfg.n_tokens):
            nb.np_step_selected(p.eng.ctx, xs[t].cuda(), B, words[t].cuda(), out, p.eng.stream, p.eng.copy_stream)
            torch.cuda.synchronize()
            res = p.ora.step(u16(xs[t]), pred_words=words[t].numpy().view(np.uint32))
            p.check_delta_against(res["deltas"])
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < REL_L2_TOL, t
            times = nb.np_last_step_times(p.eng.ctx)
            assert times[0] < 50.0                     # no predictor pass inside the call
        p.check_resident_bytes()
        with pytest.raises(nb.NpError) as e:
            nb.np_step_selected(p.eng.ctx, xs[0].cuda(), B, None, out, p.eng.stream, p.eng.copy_stream)
        assert e.value.code == nb.NP_E_INVAL
    finally:
        p.close()


def test_full_width_bank_at_7b_row_shape():
    """M = 11008, K = 512 (the paper's vocabulary) on two layers: bit-exact selection."""
    cfg = synth.StackConfig("7b2", 2, 256, 11008, 64, 10, 25, 2, 3, 0.97)
    p = Pair(cfg, max_batch=2, with_oracle=False)
    try:
        K, B, L = 512, 2, cfg.n_layers
        bank = synth.centroid_bank(cfg, K)
        z = np.random.default_rng(11).standard_normal((B, L, 2, K)).astype(np.float32)
        ids, words = _select(p, torch.from_numpy(z).cuda(), B, K, bank.cuda())
        want_ids, want_words = O.centroid_select(z, bank.numpy().view(np.uint32))
        assert (ids == want_ids).all() and (words == want_words).all()
    finally:
        p.close()
