"""Shared set-up for the GPU parity tests: one synthetic stack handed, byte for
byte, to the CUDA library and to the CPU oracle."""
import numpy as np
import torch

from oracle import np_oracle as O
from paper_2608_22643_b200 import binding as nb
from paper_2608_22643_b200 import build as nbuild
from paper_2608_22643_b200 import synth

REL_L2_TOL = 1e-3   # float outputs against the fp64 oracle (bf16 weights, fp32 accumulation)


def u16(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def rel_l2(a, b) -> float:
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a))


class Pair:
    """The CUDA engine and the oracle engine over the same bytes."""

    def __init__(self, cfg: synth.StackConfig, policy=nb.NP_EVICT_EXACT, max_batch=1, k=None, C=None,
                 transfer_mode=nb.NP_XFER_MEMCPY_RUNS, staging_rows=None, flags=nb.NP_F_CHECK_BOUNDS,
                 gen_device="cpu", with_oracle=True, chain_layers=0, ring_stages=0, dense_layers=0,
                 record_format=nb.NP_REC_BF16, store_dir=None, io_depth=0, direct=True, store_layers=0, spec_rows=0):
        nbuild.build()
        self.cfg = cfg
        self.k = cfg.top_k if k is None else k
        self.C = cfg.capacity if C is None else C
        w1, w2 = synth.predictor_weights(cfg, gen_device)
        self.w1_cpu, self.w2_cpu = w1.cpu(), w2.cpu()
        # store_layers = Lp > 0: the store holds the first Lp layers and layer l reads layer l % Lp of it
        Lp = store_layers if store_layers > 0 else cfg.n_layers
        self.backing = synth.backing_store(cfg.with_(n_layers=Lp), gen_device=gen_device)
        ncfg = nb.make_config(cfg.n_layers, cfg.d_model, cfg.d_ffn, cfg.d_pred, self.k, self.C,
                              max_batch=max_batch, evict_policy=policy, staging_rows=staging_rows,
                              transfer_mode=transfer_mode, flags=flags, chain_layers=chain_layers, ring_stages=ring_stages,
                              dense_layers=dense_layers, record_format=record_format, io_depth=io_depth,
                              store_layers=store_layers, spec_rows=spec_rows)
        self.dense_layers = dense_layers
        if record_format == nb.NP_REC_INT8:
            # the store the library reads is the 8-bit one; the oracle works on what those
            # records mean (its own dequantisation)
            self.backing_q = synth.quantize_store(self.backing)
            self.backing = self.backing_q
        if transfer_mode == nb.NP_XFER_FILE:
            # the library sees the store only as a file; the oracle keeps the bytes in memory
            path = str(store_dir / "store.bin")
            self.backing.view(torch.int16).numpy().tofile(path)
            self.eng = nb.Engine(ncfg, w1.cuda(), w2.cuda(), None, store_path=path, direct=direct)
        else:
            self.eng = nb.Engine(ncfg, w1.cuda(), w2.cuda(), self.backing)
        if record_format == nb.NP_REC_INT8:
            self.store_u16 = O.dequantize_records(self.backing_q.numpy(), cfg.d_model)
        else:
            self.store_u16 = self.backing.view(torch.int16).numpy().view(np.uint16)
        if Lp != cfg.n_layers:      # what the oracle sees: every layer's records written out
            self.store_u16 = self.store_u16[np.arange(cfg.n_layers) % Lp]
        self.ora = None
        if with_oracle:
            self.ora = O.Engine(cfg.n_layers, cfg.d_model, cfg.d_ffn, cfg.d_pred, self.k, self.C, policy,
                                u16(self.w1_cpu), u16(self.w2_cpu), self.store_u16, dense_layers=dense_layers)

    def close(self):
        self.eng.close()

    # ---- comparisons -------------------------------------------------------------------
    def check_delta_against(self, deltas):
        """Lists, counters and tables of the last np_delta are bit-identical to the oracle's."""
        cnt = self.eng.counters()
        for l, d in enumerate(deltas):
            got = self.eng.delta_lists(l, cnt[l])
            for f in ("delta_ids", "delta_slots", "evict_ids", "overflow_ids", "active_ids", "active_slots"):
                want = getattr(d, f)
                assert got[f].shape == want.shape and (got[f] == want).all(), (l, f)
            assert cnt[l][nb.NP_CNT_PRED] == d.n_pred and cnt[l][nb.NP_CNT_KEPT] == d.n_kept
            assert cnt[l][nb.NP_CNT_RESIDENT] == int(self.ora.res.R[l].sum())
            assert cnt[l][nb.NP_CNT_STEP] == self.ora.res.t - 1
            st = self.eng.export_state(l)
            # order-free validity first: a failure here is a wrong state, one below only a different order
            resident = O.bitmap_to_bool(st["resident"], self.cfg.d_ffn)
            assert O.validity_errors(st["slot_map"], st["owner"], resident, self.C) == [], l
            assert set(got["active_ids"].tolist()) <= set(np.flatnonzero(resident).tolist()), l   # act is a subset of R
            assert (st["slot_map"] == self.ora.res.S[l]).all(), l
            assert (st["owner"] == self.ora.res.owner[l]).all(), l
            assert (st["resident"] == O.bool_to_bitmap(self.ora.res.R[l])).all(), l
            assert (st["stamp"] == self.ora.res.stamp[l]).all(), l
        return cnt

    def check_resident_bytes(self):
        """Every resident row of every layer holds exactly its record's bytes."""
        torch.cuda.synchronize()
        g, u, dn = (u16(t) for t in (self.eng.gate, self.eng.up, self.eng.downT))
        nd = self.dense_layers
        for l in range(nd, self.cfg.n_layers):       # the slot buffers start at the first sparse layer
            st = self.eng.export_state(l)
            ids = np.flatnonzero(st["slot_map"] >= 0)
            slots = st["slot_map"][ids]
            assert (g[l - nd, slots] == self.store_u16[l, ids, 0]).all(), l
            assert (u[l - nd, slots] == self.store_u16[l, ids, 1]).all(), l
            assert (dn[l - nd, slots] == self.store_u16[l, ids, 2]).all(), l
        if nd:
            assert (u16(self.eng.dense) == self.store_u16[:nd]).all()
