"""Parity at the benchmark's full 7B-shaped size, in the launch configuration bench.py times
(host-gather transfer, resident multi-layer MLP kernel, default run length)."""
import numpy as np
import pytest
import torch

from oracle import np_oracle as O
from paper_2608_22643_b200 import binding as nb
from paper_2608_22643_b200 import synth
from tests.harness import REL_L2_TOL, Pair, rel_l2, u16

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("policy,mlp_flags", [(nb.NP_EVICT_EXACT, 0), (nb.NP_EVICT_LRU, 0), (nb.NP_EVICT_EXACT, nb.NP_F_CLUSTER_ROWS)])
def test_7b_shape_steps_match_oracle(policy, mlp_flags):
    cfg = synth.CONFIGS["7b"]
    L, M, D, W = cfg.n_layers, cfg.d_ffn, cfg.d_model, cfg.d_ffn // 32
    free, _ = torch.cuda.mem_get_info()
    if free < 8 * 2**30:
        pytest.skip("needs 8 GB of device memory")
    p = Pair(cfg, policy=policy, transfer_mode=nb.NP_XFER_HOST_GATHER, staging_rows=2 * cfg.top_k,
             flags=mlp_flags, gen_device="cuda")
    try:
        assert nb.np_mlp_kernel_name(p.eng.ctx, 1) == ("k_mlp_rows" if mlp_flags else "k_mlp_slices")
        n_steps = 3
        xs = synth.hidden_states(cfg, n_steps)
        logits = torch.empty((1, L, M), dtype=torch.float32, device="cuda")
        bitmap = torch.empty((L, W), dtype=torch.int32, device="cuda")
        out = torch.empty((1, D), dtype=torch.float32, device="cuda")
        rng = np.random.default_rng(0)
        w1 = O.bf16_to_f64(u16(p.w1_cpu))
        w2_u16 = u16(p.w2_cpu)
        for t in range(n_steps):
            x = xs[t].cuda()
            nb.np_predict(p.eng.ctx, x, 1, logits, bitmap, p.eng.stream)
            rc = nb.np_step(p.eng.ctx, x, 1, out, p.eng.stream, p.eng.copy_stream)
            assert rc in (nb.NP_OK, nb.NP_W_CHUNKED)
            torch.cuda.synchronize()
            z32 = logits.cpu().numpy()
            # stage 1: sampled logits, each against its own fp64 dot product
            h = np.maximum(0.0, O.bf16_to_f64(u16(xs[t])) @ w1.T)[0]
            rows = rng.integers(0, L * M, size=400)
            want = np.array([O.bf16_to_f64(w2_u16[r]) @ h for r in rows])
            got = z32.reshape(-1)[rows]
            assert np.linalg.norm(got - want) / np.linalg.norm(want) < REL_L2_TOL
            assert np.max(np.abs(got - want)) < 1e-4 * np.max(np.abs(want))
            # stage 2: the whole selection, bit-exact on the GPU's own logits
            assert (bitmap.cpu().numpy().view(np.uint32) == O.topk_bitmap(z32, p.k)).all()
            # stages 3-4 through the oracle engine (its own tables, buffers and chain)
            res = p.ora.step(u16(xs[t]), logits_f32=z32)
            cnt = p.check_delta_against(res["deltas"])
            assert (cnt[:, nb.NP_CNT_ACTIVE] == p.k).all() and (cnt[:, nb.NP_CNT_OVERFLOW] == 0).all()
            if policy == nb.NP_EVICT_EXACT:
                assert (cnt[:, nb.NP_CNT_RESIDENT] == p.k).all()
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < REL_L2_TOL, t
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < 1e-5, t
            # install: sampled resident rows of every layer hold their record's bytes
            for l in range(L):
                ids = np.flatnonzero(p.ora.res.R[l])
                pick = rng.choice(ids, size=min(48, ids.size), replace=False)
                slots = torch.from_numpy(p.ora.res.S[l][pick].astype(np.int64)).cuda()
                for part, buf in enumerate((p.eng.gate, p.eng.up, p.eng.downT)):
                    assert (u16(buf[l][slots]) == p.store_u16[l, pick, part]).all(), (t, l, part)
    finally:
        p.close()


def test_7b_long_trajectory_every_logit_and_resident_row():
    """Cold start and fifteen steady-state steps of the whole 32-layer 7B-shaped stack in the benchmark's
    launch configuration: every logit against the oracle's predictor, the whole selection, every list
    and table, every resident row of every layer byte for byte, and the chain's output, each step."""
    cfg = synth.CONFIGS["7b"]
    L, M, D, W = cfg.n_layers, cfg.d_ffn, cfg.d_model, cfg.d_ffn // 32
    free, _ = torch.cuda.mem_get_info()
    if free < 8 * 2**30:
        pytest.skip("needs 8 GB of device memory")
    p = Pair(cfg, transfer_mode=nb.NP_XFER_HOST_GATHER, staging_rows=2 * cfg.top_k, flags=0, gen_device="cuda")
    try:
        n_steps = 16
        xs = synth.hidden_states(cfg, n_steps)
        logits = torch.empty((1, L, M), dtype=torch.float32, device="cuda")
        bitmap = torch.empty((L, W), dtype=torch.int32, device="cuda")
        out = torch.empty((1, D), dtype=torch.float32, device="cuda")
        w1_u16, w2_u16 = u16(p.w1_cpu), u16(p.w2_cpu)
        for t in range(n_steps):
            x = xs[t].cuda()
            nb.np_predict(p.eng.ctx, x, 1, logits, bitmap, p.eng.stream)
            rc = nb.np_step(p.eng.ctx, x, 1, out, p.eng.stream, p.eng.copy_stream)
            assert rc in (nb.NP_OK, nb.NP_W_CHUNKED)
            torch.cuda.synchronize()
            z32 = logits.cpu().numpy()
            z = O.predict(w1_u16, w2_u16, u16(xs[t]), L, M)
            assert rel_l2(z32, z) < 1e-5 and np.max(np.abs(z32 - z)) < 1e-4 * np.max(np.abs(z)), t
            assert (bitmap.cpu().numpy().view(np.uint32) == O.topk_bitmap(z32, p.k)).all(), t
            res = p.ora.step(u16(xs[t]), logits_f32=z32)
            cnt = p.check_delta_against(res["deltas"])
            assert (cnt[:, nb.NP_CNT_ACTIVE] == p.k).all() and (cnt[:, nb.NP_CNT_OVERFLOW] == 0).all()
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < 1e-5, t
            p.check_resident_bytes()
    finally:
        p.close()


@pytest.mark.parametrize("name,n_layers,mode,chain_layers", [
    ("13b", 3, nb.NP_XFER_HOST_GATHER, 0), ("70b", 2, nb.NP_XFER_ZERO_COPY, 0), ("70b", 2, nb.NP_XFER_MEMCPY_RUNS, 0),
    # several layers per resident launch (the cross-layer hand-over of x at these row widths)
    ("13b", 4, nb.NP_XFER_HOST_GATHER, 4), ("13b", 4, nb.NP_XFER_ZERO_COPY, 2),
    ("70b", 4, nb.NP_XFER_ZERO_COPY, 4), ("70b", 4, nb.NP_XFER_HOST_GATHER, 2),
    # the row-partitioned resident kernel (the fallback of the column-sliced one) at the same widths
    ("13b", 4, nb.NP_XFER_HOST_GATHER, -4), ("70b", 4, nb.NP_XFER_ZERO_COPY, -2),
])
def test_larger_shapes_few_layers(name, n_layers, mode, chain_layers):
    """The 13B- and 70B-shaped rows (D = 5120 / 8192, M = 13824 / 28672) on a few layers:
    other ring depths, column rounds and segment splits than the 7B shape, with one and with
    several layers per resident launch."""
    cfg = synth.CONFIGS[name].with_(n_layers=n_layers)
    L, M, D, W = cfg.n_layers, cfg.d_ffn, cfg.d_model, cfg.d_ffn // 32
    flags = nb.NP_F_CHECK_BOUNDS | (nb.NP_F_ROW_CHAIN if chain_layers < 0 else 0)     # negative: the row kernel
    p = Pair(cfg, transfer_mode=mode, flags=flags, gen_device="cuda", chain_layers=abs(chain_layers))
    try:
        xs = synth.hidden_states(cfg, 3)
        logits = torch.empty((1, L, M), dtype=torch.float32, device="cuda")
        out = torch.empty((1, D), dtype=torch.float32, device="cuda")
        for t in range(3):
            x = xs[t].cuda()
            nb.np_predict(p.eng.ctx, x, 1, logits, None, p.eng.stream)
            nb.np_step(p.eng.ctx, x, 1, out, p.eng.stream, p.eng.copy_stream)
            torch.cuda.synchronize()
            z32 = logits.cpu().numpy()
            z = O.predict(u16(p.w1_cpu), u16(p.w2_cpu), u16(xs[t]), L, M)
            assert rel_l2(z32, z) < 1e-5
            res = p.ora.step(u16(xs[t]), logits_f32=z32)
            p.check_delta_against(res["deltas"])
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < 1e-5, t
        p.check_resident_bytes()
    finally:
        p.close()


@pytest.mark.parametrize("flags,kernel", [(0, "k_mlp_tc_up + k_mlp_tc_down"),
                                          (nb.NP_F_TCGEN05_BATCH, "k_mlp_up5 + k_mlp_tc_down")])
def test_stress_shape_batch16_few_layers(flags, kernel):
    """Sixteen sequences at the 7B row shape (the delta-stress workload) on four layers: the
    tensor-core predictor and the tensor-core batch MLP in the configuration bench.py --batch 16
    times (and with the up phase on tcgen05); unions of the per-sequence sets, tables bit-exact,
    chain within tolerance."""
    cfg = synth.CONFIGS["stress"].with_(n_layers=4)
    L, M, D, B = cfg.n_layers, cfg.d_ffn, cfg.d_model, 16
    p = Pair(cfg, max_batch=B, transfer_mode=nb.NP_XFER_HOST_GATHER, staging_rows=2 * cfg.top_k, flags=flags,
             gen_device="cuda")
    try:
        assert nb.np_mlp_kernel_name(p.eng.ctx, B) == kernel
        xs = synth.hidden_states(cfg, 3, batch=B, gamma=0.9)
        logits = torch.empty((B, L, M), dtype=torch.float32, device="cuda")
        out = torch.empty((B, D), dtype=torch.float32, device="cuda")
        for t in range(3):
            x = xs[t].cuda()
            nb.np_predict(p.eng.ctx, x, B, logits, None, p.eng.stream)
            rc = nb.np_step(p.eng.ctx, x, B, out, p.eng.stream, p.eng.copy_stream)
            assert rc in (nb.NP_OK, nb.NP_W_CHUNKED)
            torch.cuda.synchronize()
            z32 = logits.cpu().numpy()
            z = O.predict(u16(p.w1_cpu), u16(p.w2_cpu), u16(xs[t]), L, M)
            assert rel_l2(z32, z) < 1e-5
            res = p.ora.step(u16(xs[t]), logits_f32=z32)
            cnt = p.check_delta_against(res["deltas"])
            assert (cnt[:, nb.NP_CNT_PRED] > 1.5 * p.k).all() and (cnt[:, nb.NP_CNT_OVERFLOW] == 0).all()
            got = out.cpu().numpy()
            for b in range(B):
                assert rel_l2(got[b], res["x_final"][b]) < 1e-5, (t, b)
        p.check_resident_bytes()
    finally:
        p.close()


def test_7b_shape_with_dense_prefix():
    """The 7B row shape on six layers, the first two dense (11008 whole records each through
    the resident kernel), in bench.py's --dense-layers configuration."""
    cfg = synth.CONFIGS["7b"].with_(n_layers=6)
    L, M, D, d = cfg.n_layers, cfg.d_ffn, cfg.d_model, 2
    p = Pair(cfg, transfer_mode=nb.NP_XFER_HOST_GATHER, staging_rows=2 * cfg.top_k, flags=0, gen_device="cuda",
             dense_layers=d)
    try:
        xs = synth.hidden_states(cfg, 3)
        logits = torch.zeros((1, L, M), dtype=torch.float32, device="cuda")
        out = torch.empty((1, D), dtype=torch.float32, device="cuda")
        for t in range(3):
            x = xs[t].cuda()
            nb.np_predict(p.eng.ctx, x, 1, logits, None, p.eng.stream)
            nb.np_step(p.eng.ctx, x, 1, out, p.eng.stream, p.eng.copy_stream)
            torch.cuda.synchronize()
            z32 = logits.cpu().numpy()
            full = O.predict(u16(p.w1_cpu), u16(p.w2_cpu), u16(xs[t]), L, M).astype(np.float32)
            assert rel_l2(z32[0, d:], full[0, d:]) < 1e-5 and not z32[0, :d].any()
            full[0, d:] = z32[0, d:]
            res = p.ora.step(u16(xs[t]), logits_f32=full)
            cnt = p.check_delta_against(res["deltas"])
            assert (cnt[d:, nb.NP_CNT_ACTIVE] == p.k).all() and (cnt[:d, nb.NP_CNT_ACTIVE] == 0).all()
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < 1e-5, t
        p.check_resident_bytes()
    finally:
        p.close()
