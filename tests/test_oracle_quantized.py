"""Pins for the oracle's 8-bit record format (a transfer-path variant; the format is this
build's, its rounding is pinned against torch's own float32 -> bfloat16 conversion)."""
import numpy as np
import torch

from oracle import np_oracle as O
from paper_2608_22643_b200 import synth


def _record(q_rows, scales, D):
    rec = np.zeros(O.quantized_record_bytes(D), np.uint8)
    rec[:3 * D] = np.asarray(q_rows, np.int8).reshape(3 * D).view(np.uint8)
    rec[3 * D:3 * D + 12] = np.asarray(scales, np.float32).view(np.uint8)
    return rec


def test_layout_and_hand_values():
    D = 16
    assert O.quantized_record_bytes(4096) == 12304 and O.quantized_record_bytes(D) == 64
    q = np.zeros((3, D), np.int8)
    q[0, 0], q[0, 1], q[1, 2], q[2, 15] = 127, -127, 1, -64
    out = O.dequantize_records(_record(q, [0.5, 2.0, 0.25], D), D)
    w = O.bf16_to_f64(out)
    assert w[0, 0] == 63.5 and w[0, 1] == -63.5 and w[1, 2] == 2.0 and w[2, 15] == -16.0
    assert np.count_nonzero(w) == 4


def test_rounding_is_torchs_float32_to_bfloat16():
    # random scales make products with long mantissas; a tie is constructed as well
    rng = np.random.default_rng(0)
    D, n = 64, 200
    q = rng.integers(-127, 128, size=(n, 3, D)).astype(np.int8)
    scales = (rng.random((n, 3)).astype(np.float32) * 0.01 + 1e-4).astype(np.float32)
    scales[0, 0] = np.float32(1.0 + 2.0 ** -8)      # 1 * s = 1.00390625: exactly between two bf16 values
    q[0, 0, 0] = 1
    scales[1, 1] = np.float32(1.0 + 3 * 2.0 ** -8)  # the other tie direction (odd neighbour below)
    q[1, 1, 0] = 1
    recs = np.stack([_record(q[i], scales[i], D) for i in range(n)])
    got = O.dequantize_records(recs, D)
    prod = torch.from_numpy(q.astype(np.float32)) * torch.from_numpy(scales)[..., None]
    want = prod.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert (got == want).all()
    assert O.bf16_to_f64(got[0, 0, 0]) == 1.0 and O.bf16_to_f64(got[1, 1, 0]) == 1.015625   # ties to even


def test_quantised_store_round_trip_error_and_alignment():
    cfg = synth.CONFIGS["tiny"]
    store = synth.backing_store(cfg)
    qs = synth.quantize_store(store)
    assert qs.shape == (cfg.n_layers, cfg.d_ffn, O.quantized_record_bytes(cfg.d_model)) and qs.shape[-1] % 16 == 0
    deq = O.bf16_to_f64(O.dequantize_records(qs.numpy(), cfg.d_model))
    ref = store.to(torch.float64).numpy()
    # symmetric 8-bit rows: at most half a step of the row's scale, plus the bf16 rounding
    step = np.abs(ref).max(axis=-1, keepdims=True) / 127.0
    assert (np.abs(deq - ref) <= 0.5 * step + np.abs(ref) * 2.0 ** -8 + 1e-12).all()
    assert np.abs(deq - ref).max() > 0          # it is a different store
