"""GPU parity: every stage of the CUDA path against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import np_oracle as O
from paper_2608_22643_b200 import binding as nb
from paper_2608_22643_b200 import synth
from tests.harness import REL_L2_TOL, Pair, rel_l2, u16

pytestmark = pytest.mark.gpu

TINY = synth.CONFIGS["tiny"]
SMALL = synth.CONFIGS["small"]     # ragged: M = 2080 (65 words), H = 96, 3 layers


# predictor width a multiple of 64 (three k-blocks) and a row count that is not a multiple of
# the 128-row MMA tile: the batch path runs on the tensor cores with a ragged last tile
TCW = synth.StackConfig("tcw", 3, 512, 2080, 192, 10, 25, 4, 21, 0.9)
# predictor width a multiple of the 128-row MMA tile: layer 1 of a batch runs on the tensor cores too (one K range
# per block at D = 512, sixteen ranges of four K blocks at D = 4096, a ragged last range at D = 4160)
TC1 = synth.StackConfig("tc1", 2, 512, 1024, 128, 10, 25, 4, 22, 0.9)
TC1W = synth.StackConfig("tc1w", 2, 4096, 1024, 256, 10, 25, 4, 23, 0.9)
TC1R = synth.StackConfig("tc1r", 2, 4160, 1024, 384, 10, 25, 4, 24, 0.9)


@pytest.mark.parametrize("cfg,B,flags", [
    (TINY, 1, 0), (SMALL, 1, 0), (SMALL, 3, 0), (TINY, 16, 0), (TCW, 16, 0), (TCW, 7, 0), (TCW, 5, 0),
    (TCW, 16, nb.NP_F_NO_TENSOR_CORES), (SMALL, 9, 0),
    (TC1, 5, 0), (TC1, 16, 0), (TC1W, 16, 0), (TC1W, 9, 0), (TC1R, 16, 0), (TC1R, 6, 0),
])
def test_predict_logits_and_bitmap(cfg, B, flags):
    p = Pair(cfg, max_batch=B, flags=flags | nb.NP_F_CHECK_BOUNDS)
    try:
        xs = synth.hidden_states(cfg, 3, batch=B)
        L, M, W = cfg.n_layers, cfg.d_ffn, cfg.d_ffn // 32
        logits = torch.empty((B, L, M), dtype=torch.float32, device="cuda")
        bitmap = torch.empty((L, W), dtype=torch.int32, device="cuda")
        for t in range(3):
            x = xs[t].cuda()
            nb.np_predict(p.eng.ctx, x, B, logits, bitmap, p.eng.stream)
            p.eng.stream.synchronize()
            z = O.predict(u16(p.w1_cpu), u16(p.w2_cpu), u16(xs[t]), L, M)
            assert rel_l2(logits.cpu().numpy(), z) < REL_L2_TOL
            assert rel_l2(logits.cpu().numpy(), z) < 1e-5      # fp32 accumulation does far better
            # selection is verified on the GPU's own logits: bit-exact
            want = O.topk_bitmap(logits.cpu().numpy(), p.k)
            got = bitmap.cpu().numpy().view(np.uint32)
            assert (got == want).all()
    finally:
        p.close()


def _topk_case(p, z):
    B, L, M = z.shape
    out = torch.empty((L, M // 32), dtype=torch.int32, device="cuda")
    nb.np_topk(p.eng.ctx, torch.from_numpy(z).cuda(), B, out, p.eng.stream)
    p.eng.stream.synchronize()
    assert (out.cpu().numpy().view(np.uint32) == O.topk_bitmap(z, p.k)).all()


def test_topk_edge_cases():
    cfg = TINY
    L, M = cfg.n_layers, cfg.d_ffn
    rng = np.random.default_rng(0)
    p = Pair(cfg, max_batch=4, with_oracle=False)
    try:
        _topk_case(p, np.zeros((1, L, M), np.float32))                       # all equal -> lowest indices
        z = np.full((1, L, M), -0.0, np.float32); z[:, :, 500:600:7] = 0.0   # +0 above -0
        _topk_case(p, z)
        _topk_case(p, -np.abs(rng.standard_normal((1, L, M))).astype(np.float32))   # all negative
        z = rng.standard_normal((1, L, M)).astype(np.float32)
        z[:, :, ::3] = z[:, :, 1:2]                                          # a third of the keys tie
        _topk_case(p, z)
        z = rng.integers(-3, 4, size=(4, L, M)).astype(np.float32)           # heavy ties, batch union
        _topk_case(p, z)
        z = rng.standard_normal((2, L, M)).astype(np.float32) * 1e30
        z[0, 0, 5] = np.inf; z[1, 1, 7] = -np.inf; z[0, 1, 9] = 1e-42        # inf and a denormal
        _topk_case(p, z)
    finally:
        p.close()
    for k, C in ((0, 8), (M, M), (1, 1)):                                    # degenerate k
        p = Pair(cfg, k=k, C=C, with_oracle=False)
        try:
            _topk_case(p, rng.standard_normal((1, L, M)).astype(np.float32))
        finally:
            p.close()


def test_topk_paths_of_the_selection_kernel():
    """The selection kernel bins the logits linearly and ranks the deciding bin directly; ranges, ties and
    clusters that it has to hand to its general (radix) path, and the boundary between the two."""
    cfg = TINY.with_(d_ffn=4096)
    L, M = cfg.n_layers, cfg.d_ffn
    rng = np.random.default_rng(5)
    p = Pair(cfg, with_oracle=False)
    try:
        k = p.k
        assert 300 < k < 1000
        z = rng.standard_normal((1, L, M)).astype(np.float32)
        z[:, :, 7] = 3e38; z[:, :, 9] = -3e38                               # max - min overflows
        _topk_case(p, z)
        for n_tie in (1024, 1025, 2000):                                    # n_tie equal keys around the k-th place
            z = rng.standard_normal((1, L, M)).astype(np.float32)
            order = np.argsort(-z[0], axis=1)
            for l in range(L):
                v = z[0, l, order[l, k]]
                idx = rng.permutation(order[l, k - 200:k - 200 + n_tie])    # 200 of them above the cut, the rest below
                z[0, l, idx] = v
            _topk_case(p, z)
        z = (1.0 + rng.permutation(M)[None, None, :].repeat(L, 1) * 2.0**-23).astype(np.float32)   # consecutive floats
        _topk_case(p, z)
        z = rng.standard_normal((1, L, M)).astype(np.float32) * 1e-3        # two far clusters, the cut inside the lower one
        z[:, :, :200] += 1e6
        _topk_case(p, z)
        z = rng.standard_normal((1, L, M)).astype(np.float32) * 1e-42       # denormals only
        _topk_case(p, z)
        z = np.where(rng.random((1, L, M)) < 0.5, -0.0, 0.0).astype(np.float32)   # signed zeros only
        _topk_case(p, z)
    finally:
        p.close()


@pytest.mark.parametrize("policy", [nb.NP_EVICT_EXACT, nb.NP_EVICT_LRU])
@pytest.mark.parametrize("cfg,n_set,C,persist", [
    (TINY, 102, 205, 0.8), (TINY, 102, 102, 0.6), (SMALL, 208, 520, 0.83), (SMALL, 700, 520, 0.7),
    (TINY, 1, 1, 0.0), (TINY, 0, 4, 0.5),
    (TINY.with_(d_ffn=12288), 5000, 6000, 0.3), (TINY.with_(d_ffn=12288), 7000, 6000, 0.3),
])
def test_delta_lists_and_tables_bit_exact(policy, cfg, n_set, C, persist):
    """Injected bitmap sequences (fixed-size sets, full replacement, oversize sets that
    overflow capacity, the empty set, lists of several thousand rows: longer than what the
    kernel keeps in shared memory) against the oracle, every step."""
    T = 10
    p = Pair(cfg, policy=policy, k=min(n_set, C), C=C)
    try:
        words = synth.random_bitmaps(cfg.n_layers, cfg.d_ffn, n_set, 11, T, persist)
        for t in range(T):
            nb.np_delta(p.eng.ctx, words[t].cuda(), p.eng.stream)
            deltas = p.ora.res.delta(words[t].numpy().view(np.uint32))
            cnt = p.check_delta_against(deltas)
            rc = nb.np_install(p.eng.ctx, 0, cfg.n_layers, p.eng.copy_stream)
            if n_set > C:
                assert rc == nb.NP_W_OVERFLOW and (cnt[:, nb.NP_CNT_OVERFLOW] > 0).all()
            for l, d in enumerate(deltas):
                O.install(p.store_u16, p.ora.gate, p.ora.up, p.ora.downT, l, d.delta_ids, d.delta_slots)
        p.check_resident_bytes()
    finally:
        p.close()


@pytest.mark.parametrize("mode,staging_rows", [
    (nb.NP_XFER_MEMCPY_RUNS, None), (nb.NP_XFER_MEMCPY_RUNS, 1), (nb.NP_XFER_MEMCPY_RUNS, 7),
    (nb.NP_XFER_HOST_GATHER, None), (nb.NP_XFER_HOST_GATHER, 2), (nb.NP_XFER_HOST_GATHER, 9),
    (nb.NP_XFER_ZERO_COPY, None),
])
def test_install_every_transfer_mode_and_chunking(mode, staging_rows):
    """After each step every resident row holds its record's bytes, however the
    delta was moved and however small the staging buffer is (Section 3.5)."""
    cfg = SMALL
    p = Pair(cfg, transfer_mode=mode, staging_rows=staging_rows)
    try:
        words = synth.random_bitmaps(cfg.n_layers, cfg.d_ffn, p.k, 5, 6, 0.8)
        # make some IDs adjacent so that run coalescing has work to do
        words[:, :, 3] = -1
        for t in range(6):
            nb.np_delta(p.eng.ctx, words[t].cuda(), p.eng.stream)
            rc = nb.np_install(p.eng.ctx, 0, cfg.n_layers, p.eng.copy_stream)
            if staging_rows is not None and mode != nb.NP_XFER_ZERO_COPY and t == 0:
                assert rc == nb.NP_W_CHUNKED
            p.check_resident_bytes()
            deltas = p.ora.res.delta(words[t].numpy().view(np.uint32))
            p.check_delta_against(deltas)
    finally:
        p.close()


@pytest.mark.parametrize("cfg,B", [(TINY, 1), (SMALL, 1), (SMALL, 2), (SMALL, 5)])
def test_sparse_mlp_per_layer(cfg, B):
    p = Pair(cfg, max_batch=B)
    try:
        words = synth.random_bitmaps(cfg.n_layers, cfg.d_ffn, p.k, 9, 3, 0.8)
        rng = np.random.default_rng(4)
        for t in range(3):
            nb.np_delta(p.eng.ctx, words[t].cuda(), p.eng.stream)
            nb.np_install(p.eng.ctx, 0, cfg.n_layers, p.eng.copy_stream)
            deltas = p.ora.res.delta(words[t].numpy().view(np.uint32))
            for l, d in enumerate(deltas):
                O.install(p.store_u16, p.ora.gate, p.ora.up, p.ora.downT, l, d.delta_ids, d.delta_slots)
            x = rng.standard_normal((B, cfg.d_model)).astype(np.float32)
            xd = torch.from_numpy(x).cuda()
            y = torch.full((B, cfg.d_model), 7.0, dtype=torch.float32, device="cuda")   # must be overwritten
            for l, d in enumerate(deltas):
                nb.np_sparse_mlp(p.eng.ctx, l, xd, B, y, p.eng.stream)
                p.eng.stream.synchronize()
                want = O.sparse_mlp(p.ora.gate, p.ora.up, p.ora.downT, l, d.active_slots, x.astype(np.float64))
                assert rel_l2(y.cpu().numpy(), want) < REL_L2_TOL, (t, l)
                assert rel_l2(y.cpu().numpy(), want) < 1e-5, (t, l)
    finally:
        p.close()


def test_all_rows_active_is_the_dense_mlp():
    """k = C = M: the sparse path over every row equals the dense SwiGLU MLP."""
    cfg = TINY
    M = cfg.d_ffn
    p = Pair(cfg, k=M, C=M)
    try:
        x_bf = synth.hidden_states(cfg, 1)[0]
        out = torch.empty((1, cfg.d_model), dtype=torch.float32, device="cuda")
        nb.np_step(p.eng.ctx, x_bf.cuda(), 1, out, p.eng.stream, p.eng.copy_stream)
        torch.cuda.synchronize()
        x = x_bf.to(torch.float64)
        for l in range(cfg.n_layers):
            rec = p.backing[l].to(torch.float64)
            n = x / torch.sqrt((x * x).mean(dim=-1, keepdim=True) + 1e-6)     # pre-MLP RMS norm, unit gain
            x = x + (torch.nn.functional.silu(n @ rec[:, 0].T) * (n @ rec[:, 1].T)) @ rec[:, 2]
        assert rel_l2(out.cpu().numpy(), x.numpy()) < REL_L2_TOL
    finally:
        p.close()


@pytest.mark.parametrize("policy", [nb.NP_EVICT_EXACT, nb.NP_EVICT_LRU])
@pytest.mark.parametrize("mode", [nb.NP_XFER_MEMCPY_RUNS, nb.NP_XFER_HOST_GATHER, nb.NP_XFER_ZERO_COPY])
@pytest.mark.parametrize("cfg,B", [(TINY, 1), (SMALL, 4)])
def test_whole_step_trajectory(policy, mode, cfg, B):
    """np_step over the config's token sequence: selection bit-exact on the GPU's own
    logits, lists/tables bit-exact, chain output within tolerance, state carried."""
    p = Pair(cfg, policy=policy, transfer_mode=mode, max_batch=B, C=cfg.capacity if B == 1 else cfg.d_ffn // 2)
    try:
        xs = synth.hidden_states(cfg, cfg.n_tokens, batch=B)
        L, M, W = cfg.n_layers, cfg.d_ffn, cfg.d_ffn // 32
        out = torch.empty((B, cfg.d_model), dtype=torch.float32, device="cuda")
        logits = torch.empty((B, L, M), dtype=torch.float32, device="cuda")
        for t in range(cfg.n_tokens):
            # the predictor kernels are deterministic: this call's logits are the step's logits
            nb.np_predict(p.eng.ctx, xs[t].cuda(), B, logits, None, p.eng.stream)
            nb.np_step(p.eng.ctx, xs[t].cuda(), B, out, p.eng.stream, p.eng.copy_stream)
            torch.cuda.synchronize()
            z32 = logits.cpu().numpy()
            res = p.ora.step(u16(xs[t]), logits_f32=z32)
            p.check_delta_against(res["deltas"])
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < REL_L2_TOL, t
            # informational: the oracle's own logits agree with the GPU's
            z = O.predict(u16(p.w1_cpu), u16(p.w2_cpu), u16(xs[t]), L, M)
            assert rel_l2(z32, z) < 1e-5
        p.check_resident_bytes()
        us = nb.np_last_step_times(p.eng.ctx)
        assert (us >= 0).all()
    finally:
        p.close()


# a stack whose per-block share (k = 900 rows over the SMs) exceeds a small ring several times
# over, so that shared-memory stages are reused within a layer and across layers
DENSE = synth.StackConfig("dense", 4, 512, 2048, 64, 44, 60, 5, 13, 0.9)


@pytest.mark.parametrize("flags,chain_layers,ring_stages", [
    (nb.NP_F_CHECK_BOUNDS, 1, 0), (nb.NP_F_CHECK_BOUNDS, 2, 0), (nb.NP_F_CHECK_BOUNDS, 0, 0), (0, 0, 0),
    (nb.NP_F_CHECK_BOUNDS, 0, 2), (nb.NP_F_CHECK_BOUNDS, 3, 3), (nb.NP_F_CHECK_BOUNDS, 0, 4),
    (nb.NP_F_CHECK_BOUNDS | nb.NP_F_ROW_CHAIN, 0, 0), (nb.NP_F_CHECK_BOUNDS | nb.NP_F_ROW_CHAIN, 2, 3),
    (nb.NP_F_CHECK_BOUNDS | nb.NP_F_LAYER_LAUNCHES, 0, 0),
    (nb.NP_F_CHECK_BOUNDS | nb.NP_F_LAYER_LAUNCHES, 0, 2),
    (nb.NP_F_CHECK_BOUNDS | nb.NP_F_LAYER_LAUNCHES, 0, 5),
    (nb.NP_F_CHECK_BOUNDS | nb.NP_F_LAYER_LAUNCHES | nb.NP_F_DIRECT_LOADS, 0, 0),
])
@pytest.mark.parametrize("cfg", [TINY, SMALL, DENSE])
def test_mlp_kernel_variants_agree_with_oracle(cfg, flags, chain_layers, ring_stages):
    """The resident multi-layer kernel (any run length), the staged per-layer kernel and the
    direct-load kernel all reproduce the oracle's residual chain."""
    p = Pair(cfg, flags=flags, chain_layers=chain_layers, ring_stages=ring_stages)
    try:
        xs = synth.hidden_states(cfg, 5)
        L, M = cfg.n_layers, cfg.d_ffn
        out = torch.empty((1, cfg.d_model), dtype=torch.float32, device="cuda")
        logits = torch.empty((1, L, M), dtype=torch.float32, device="cuda")
        for t in range(5):
            nb.np_predict(p.eng.ctx, xs[t].cuda(), 1, logits, None, p.eng.stream)
            nb.np_step(p.eng.ctx, xs[t].cuda(), 1, out, p.eng.stream, p.eng.copy_stream)
            torch.cuda.synchronize()
            res = p.ora.step(u16(xs[t]), logits_f32=logits.cpu().numpy())
            p.check_delta_against(res["deltas"])
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < 1e-5, t
            # the chain alone, on the state the step left behind, gives the same vector
            out2 = torch.empty_like(out)
            nb.np_mlp_chain(p.eng.ctx, xs[t].cuda(), 1, out2, p.eng.stream)
            p.eng.stream.synchronize()
            assert rel_l2(out2.cpu().numpy(), res["x_final"]) < 1e-5, t
    finally:
        p.close()


@pytest.mark.parametrize("flags", [nb.NP_F_CHECK_BOUNDS, nb.NP_F_CHECK_BOUNDS | nb.NP_F_LAYER_LAUNCHES])
@pytest.mark.parametrize("n_set", [0, 1, 100, 1200])
def test_resident_chain_with_set_sizes_away_from_k(n_set, flags):
    """Active sets the caller supplies, from empty to nearly the whole capacity: blocks without
    rows, and shares of more rows than one tile holds (the kernels were planned for k rows)."""
    cfg = DENSE
    p = Pair(cfg, flags=flags)
    try:
        L, D = cfg.n_layers, cfg.d_model
        assert n_set <= p.C
        words = synth.random_bitmaps(L, cfg.d_ffn, max(n_set, 1), 77, 3, 0.6)
        if n_set == 0:
            words.zero_()
        xs = synth.hidden_states(cfg, 3)
        out = torch.empty((1, D), dtype=torch.float32, device="cuda")
        for t in range(3):
            nb.np_step_selected(p.eng.ctx, xs[t].cuda(), 1, words[t].cuda(), out, p.eng.stream, p.eng.copy_stream)
            torch.cuda.synchronize()
            res = p.ora.step(u16(xs[t]), pred_words=words[t].numpy().view(np.uint32))
            p.check_delta_against(res["deltas"])
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < 1e-5, t
        p.eng.counters()
    finally:
        p.close()


def test_chain_in_one_launch_is_reproducible_bit_for_bit():
    """On resident rows the whole stack is one resident launch, its sums between layers and behind the last one
    are integer adds (which commute) and the exchange adds its four slices in a fixed order: the result does not
    depend on the order in which the blocks arrive, so repeated calls give the same bits."""
    cfg = DENSE
    p = Pair(cfg, chain_layers=cfg.n_layers)
    try:
        assert nb.np_mlp_kernel_name(p.eng.ctx, 1) == "k_mlp_slices"
        xs = synth.hidden_states(cfg, 2)
        out = torch.empty((1, cfg.d_model), dtype=torch.float32, device="cuda")
        logits = torch.empty((1, cfg.n_layers, cfg.d_ffn), dtype=torch.float32, device="cuda")
        nb.np_predict(p.eng.ctx, xs[0].cuda(), 1, logits, None, p.eng.stream)
        nb.np_step(p.eng.ctx, xs[0].cuda(), 1, out, p.eng.stream, p.eng.copy_stream)
        torch.cuda.synchronize()
        res = p.ora.step(u16(xs[0]), logits_f32=logits.cpu().numpy())
        runs = []
        for _ in range(6):
            o = torch.empty_like(out)
            nb.np_mlp_chain(p.eng.ctx, xs[0].cuda(), 1, o, p.eng.stream)
            torch.cuda.synchronize()
            assert nb.np_chain_launches(p.eng.ctx) == 1
            runs.append(o.cpu().numpy())
        assert rel_l2(runs[0], res["x_final"]) < 1e-5
        for o in runs[1:]:
            assert (o.view(np.uint32) == runs[0].view(np.uint32)).all()
        p.eng.counters()
    finally:
        p.close()


def test_partial_sums_beyond_the_counted_words_range_are_reported():
    """Between the layers of a launch the resident kernel hands the MLP's partial sums over as counted
    fixed-point words (|sum| < 2^19 per block).  Down rows of 3e6 push layer 0 far past that: the launch
    must say so in the status word (bit 16), not hand on a wrapped sum."""
    cfg = DENSE
    p = Pair(cfg, with_oracle=False, chain_layers=cfg.n_layers)
    try:
        assert nb.np_mlp_kernel_name(p.eng.ctx, 1) == "k_mlp_slices"
        p.backing[0, :, 2, :] = 3.0e6                       # record = [gate | up | down] vectors of a neuron
        words = synth.random_bitmaps(cfg.n_layers, cfg.d_ffn, p.k, 3, 1, 0.6)
        x = synth.hidden_states(cfg, 1)[0].cuda()
        out = torch.empty((1, cfg.d_model), dtype=torch.float32, device="cuda")
        nb.np_step_selected(p.eng.ctx, x, 1, words[0].cuda(), out, p.eng.stream, p.eng.copy_stream)
        torch.cuda.synchronize()
        with pytest.raises(nb.NpError, match="0x10"):
            p.eng.counters()
    finally:
        p.close()


def test_call_order_and_argument_errors():
    p = Pair(TINY, with_oracle=False)
    try:
        ctx = p.eng.ctx
        lib = nb.load()
        assert lib.np_install(ctx, 0, 1, None) == nb.NP_E_STATE          # no delta yet
        assert lib.np_delta(ctx, None, None) == nb.NP_E_STATE            # no predict yet
        y = torch.zeros(256, device="cuda")
        assert lib.np_sparse_mlp(ctx, 0, y.data_ptr(), 1, y.data_ptr(), None) == nb.NP_E_STATE
        assert lib.np_sparse_mlp(ctx, 5, y.data_ptr(), 1, y.data_ptr(), None) == nb.NP_E_INVAL
        assert lib.np_predict(ctx, y.data_ptr(), 2, None, None, None) == nb.NP_E_INVAL   # B > max_batch
        assert lib.np_install(ctx, 1, 0, None) == nb.NP_E_INVAL
        assert "np_install" in nb.np_last_error(ctx) or "layer" in nb.np_last_error(ctx)
        words = synth.random_bitmaps(2, 1024, 50, 1, 1)
        nb.np_delta(ctx, words[0].cuda(), p.eng.stream)
        assert nb.np_install(ctx, 0, 2, p.eng.copy_stream) == nb.NP_OK
        nb.np_reset(ctx, p.eng.stream)
        assert lib.np_install(ctx, 0, 1, None) == nb.NP_E_STATE
        st = p.eng.export_state(0)
        assert (st["slot_map"] == -1).all() and (st["owner"] == -1).all() and not st["resident"].any()
    finally:
        p.close()


def test_export_import_roundtrip_resumes_trajectory():
    cfg = TINY
    a = Pair(cfg, policy=nb.NP_EVICT_LRU)
    b = Pair(cfg, policy=nb.NP_EVICT_LRU, with_oracle=False)
    try:
        words = synth.random_bitmaps(cfg.n_layers, cfg.d_ffn, a.k, 21, 8, 0.7)
        for t in range(4):
            nb.np_delta(a.eng.ctx, words[t].cuda(), a.eng.stream)
            a.ora.res.delta(words[t].numpy().view(np.uint32))
        for l in range(cfg.n_layers):
            st = a.eng.export_state(l)
            nb.np_import_state(b.eng.ctx, l, st["slot_map"], st["owner"], st["resident"], st["stamp"], 4,
                               b.eng.stream)
        for t in range(4, 8):
            nb.np_delta(b.eng.ctx, words[t].cuda(), b.eng.stream)
            deltas = a.ora.res.delta(words[t].numpy().view(np.uint32))
            b.ora = a.ora
            b.check_delta_against(deltas)
    finally:
        a.close()
        b.close()


@pytest.mark.parametrize("H", [16, 24, 40, 136, 264, 520, 1024, 1032])
@pytest.mark.parametrize("L,M", [(1, 32), (2, 96), (3, 1024)])
def test_predictor_widths_and_row_counts(H, L, M):
    """Hidden widths on both sides of every lane-layout boundary of the layer-2 kernels, with
    fewer rows than blocks, a row or two per block, and many."""
    cfg = synth.StackConfig("pw", L, 64, M, H, 25, 50, 2, 41, 0.9)
    for B in (1, 2):
        p = Pair(cfg, max_batch=B, with_oracle=False)
        try:
            xs = synth.hidden_states(cfg, 2, batch=B)
            logits = torch.full((B, L, M), 7.0, dtype=torch.float32, device="cuda")
            for t in range(2):
                nb.np_predict(p.eng.ctx, xs[t].cuda(), B, logits, None, p.eng.stream)
                p.eng.stream.synchronize()
                z = O.predict(u16(p.w1_cpu), u16(p.w2_cpu), u16(xs[t]), L, M)
                assert rel_l2(logits.cpu().numpy(), z) < 1e-5, (B, t)
            p.eng.counters()
        finally:
            p.close()


@pytest.mark.parametrize("shape", [
    # name, L, D, M, H, density %, capacity %
    ("max_ffn", 1, 64, 40960, 8, 10, 20),        # widest FFN the library accepts (top-k keys fill shared memory)
    ("max_model", 2, 16384, 64, 64, 25, 50),     # widest model: 96 KB records, four column rounds
    ("max_pred", 2, 64, 64, 4096, 25, 50),       # widest predictor: 8 KB rows of W2
    ("min_all", 1, 8, 32, 8, 10, 20),            # smallest legal sizes
])
@pytest.mark.parametrize("B", [1, 3])
def test_limit_shapes(shape, B, chain_layers=0):
    """The extreme sizes np_init accepts run the whole path and match the oracle."""
    name, L, D, M, H, dens, cap = shape
    cfg = synth.StackConfig(name, L, D, M, H, dens, cap, 3, 31, 0.9)
    p = Pair(cfg, max_batch=B, k=max(1, cfg.top_k), C=max(2, cfg.capacity), chain_layers=chain_layers)
    try:
        xs = synth.hidden_states(cfg, 3, batch=B)
        out = torch.empty((B, D), dtype=torch.float32, device="cuda")
        logits = torch.empty((B, L, M), dtype=torch.float32, device="cuda")
        for t in range(3):
            nb.np_predict(p.eng.ctx, xs[t].cuda(), B, logits, None, p.eng.stream)
            nb.np_step(p.eng.ctx, xs[t].cuda(), B, out, p.eng.stream, p.eng.copy_stream)
            torch.cuda.synchronize()
            z32 = logits.cpu().numpy()
            assert rel_l2(z32, O.predict(u16(p.w1_cpu), u16(p.w2_cpu), u16(xs[t]), L, M)) < 1e-5
            res = p.ora.step(u16(xs[t]), logits_f32=z32)
            p.check_delta_against(res["deltas"])
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < 1e-5, t
        p.check_resident_bytes()
    finally:
        p.close()


@pytest.mark.parametrize("chain_layers", [2, 4])
def test_widest_model_with_several_layers_per_launch(chain_layers):
    """D = 16384 on four layers, two and four of them per resident launch: x is handed from
    layer to layer inside the kernel at the widest row the library accepts."""
    test_limit_shapes(("max_model_chain", 4, 16384, 64, 64, 25, 50), 1, chain_layers=chain_layers)


@pytest.mark.parametrize("D,M,L,chain_layers,dense,policy", [
    (1024, 4096, 5, 0, 0, nb.NP_EVICT_EXACT),     # three rows a block, all layers in one launch
    (2048, 2048, 4, 2, 0, nb.NP_EVICT_LRU),       # x handed from launch to launch
    (4096, 4096, 3, 1, 0, nb.NP_EVICT_EXACT),     # the 7B row width, a launch per layer
    (1024, 16384, 3, 0, 0, nb.NP_EVICT_EXACT),    # eleven rows a block: two MMA row blocks, two batches of tensor-memory reads
    (1024, 4096, 5, 0, 2, nb.NP_EVICT_EXACT),     # behind a dense prefix: the run starts from another kernel's hand-over
])
def test_cluster_rows_kernel(D, M, L, chain_layers, dense, policy):
    """NP_F_CLUSTER_ROWS: whole rows per block, blocks in clusters that reduce among themselves through distributed
    shared memory, down rows parked in tensor memory.  The whole step against the oracle, every step."""
    cfg = synth.StackConfig("cluster_rows", L, D, M, 64, 10, 25, 4, 77, 0.9)
    p = Pair(cfg, policy=policy, flags=nb.NP_F_CHECK_BOUNDS | nb.NP_F_CLUSTER_ROWS, chain_layers=chain_layers, dense_layers=dense)
    try:
        assert nb.np_mlp_kernel_name(p.eng.ctx, 1) == "k_mlp_rows"
        xs = synth.hidden_states(cfg, 4)
        out = torch.empty((1, D), dtype=torch.float32, device="cuda")
        logits = torch.empty((1, L, M), dtype=torch.float32, device="cuda")
        for t in range(4):
            nb.np_predict(p.eng.ctx, xs[t].cuda(), 1, logits, None, p.eng.stream)
            nb.np_step(p.eng.ctx, xs[t].cuda(), 1, out, p.eng.stream, p.eng.copy_stream)
            torch.cuda.synchronize()
            res = p.ora.step(u16(xs[t]), logits_f32=logits.cpu().numpy())
            p.check_delta_against(res["deltas"])
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < 1e-5, t
        # the chain alone, twice: the kernel's counters and accumulators carry over from launch to launch
        for _ in range(2):
            nb.np_mlp_chain(p.eng.ctx, xs[3].cuda(), 1, out, p.eng.stream)
            torch.cuda.synchronize()
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < 1e-5
        p.eng.counters()    # reading the counters also checks the status word
    finally:
        p.close()


@pytest.mark.parametrize("mode,dense", [(nb.NP_XFER_MEMCPY_RUNS, 0), (nb.NP_XFER_HOST_GATHER, 0), (nb.NP_XFER_ZERO_COPY, 0),
                                        (nb.NP_XFER_HOST_GATHER, 3), (nb.NP_XFER_FILE, 0), (nb.NP_XFER_FILE, 3)])
def test_store_aliased_over_fewer_layers(mode, dense, tmp_path):
    """store_layers = 2 on a five-layer stack: layer l reads the records of layer l mod 2 (a stack whose
    whole store the host cannot hold), through every transfer mode and through a dense prefix that
    wraps around the store; the oracle is handed the five layers written out."""
    cfg = SMALL.with_(n_layers=5)
    p = Pair(cfg, transfer_mode=mode, store_layers=2, dense_layers=dense, store_dir=tmp_path)
    try:
        assert p.backing.shape[0] == 2
        xs = synth.hidden_states(cfg, 4)
        L, M = cfg.n_layers, cfg.d_ffn
        out = torch.empty((1, cfg.d_model), dtype=torch.float32, device="cuda")
        logits = torch.zeros((1, L, M), dtype=torch.float32, device="cuda")
        for t in range(4):
            nb.np_predict(p.eng.ctx, xs[t].cuda(), 1, logits, None, p.eng.stream)
            nb.np_step(p.eng.ctx, xs[t].cuda(), 1, out, p.eng.stream, p.eng.copy_stream)
            torch.cuda.synchronize()
            res = p.ora.step(u16(xs[t]), logits_f32=logits.cpu().numpy())
            p.check_delta_against(res["deltas"])
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < 1e-5, t
        p.check_resident_bytes()
    finally:
        p.close()


def test_bounded_wait_times_out_and_context_survives():
    """A wait that nothing satisfies gives up, is reported as NP_E_DEVICE, and after np_reset
    the context computes correctly again (no hang, no trap)."""
    p = Pair(TINY)
    try:
        assert nb.np_selftest_bounded_wait(p.eng.ctx, p.eng.stream) == nb.NP_E_DEVICE
        assert "bounds check" in nb.np_last_error(p.eng.ctx) or "status" in nb.np_last_error(p.eng.ctx)
        with pytest.raises(nb.NpError):
            p.eng.counters()                      # the status word stays set ...
        nb.np_reset(p.eng.ctx, p.eng.stream)      # ... until the context is reset
        xs = synth.hidden_states(TINY, 2)
        out = torch.empty((1, TINY.d_model), dtype=torch.float32, device="cuda")
        logits = torch.empty((1, TINY.n_layers, TINY.d_ffn), dtype=torch.float32, device="cuda")
        for t in range(2):
            nb.np_predict(p.eng.ctx, xs[t].cuda(), 1, logits, None, p.eng.stream)
            nb.np_step(p.eng.ctx, xs[t].cuda(), 1, out, p.eng.stream, p.eng.copy_stream)
            torch.cuda.synchronize()
            res = p.ora.step(u16(xs[t]), logits_f32=logits.cpu().numpy())
            p.check_delta_against(res["deltas"])
            assert rel_l2(out.cpu().numpy(), res["x_final"]) < 1e-5
    finally:
        p.close()
