"""Seeded synthetic workloads shaped like the paper's MLP stacks.

This module only draws random numbers and lays bytes out; it contains none of
the method's arithmetic (no predictor, selection, residency or MLP math), so
the CPU oracle and the CUDA path can both be fed from it without sharing code.

Everything is handed out as raw bf16 bit patterns (``torch.bfloat16`` tensors,
or ``uint16`` views of them): those bytes are the ground truth both sides read.

Recipe
------
* Weights: one ``torch.Generator`` per tensor, seeded with
  ``seed * 1_000_003 + tensor_id``; ``randn * 0.02`` rounded to bf16.
  ``tensor_id``: 0 = W1 ``[H, D]``, 1 = W2 ``[L*M, H]``, ``2 + l`` = the
  neuron-centric record block of layer ``l``, ``[M, 3, D]`` with the three rows
  of a record being gate, up and transposed-down (the layer-major repacked
  layout of Section 3.5 of the paper, with a pinned-host array standing in for
  the NVMe file).
* Hidden states: ``x_0 ~ N(0, I)``, ``x_t = rho * x_{t-1} + sqrt(1 - rho^2) *
  eps_t`` in fp32 (generator seeded ``seed * 1_000_003 + 999``), rounded to
  bf16.  For batches, every sequence mixes one shared AR(1) driver with its own
  AR(1) process: ``x^(b) = sqrt(gamma) * s + sqrt(1 - gamma) * u^(b)``.

The paper's own activations (Mistral-7B / Llama-3-8B on WikiText-2 and
HellaSwag) are not available; these inputs stand in for them and reproduce only
the shapes and the token-to-token persistence statistic.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import torch

_SEED_MUL = 1_000_003


@dataclasses.dataclass(frozen=True)
class StackConfig:
    """Shapes of one synthetic MLP stack (notation: L, D, M, H, k, C)."""

    name: str
    n_layers: int      # L
    d_model: int       # D
    d_ffn: int         # M
    d_pred: int        # H
    density_pct: int   # top-k density, percent of M
    capacity_pct: int  # resident capacity, percent of M
    n_tokens: int
    seed: int
    rho: float

    @property
    def top_k(self) -> int:
        return (self.density_pct * self.d_ffn + 50) // 100

    @property
    def capacity(self) -> int:
        return (self.capacity_pct * self.d_ffn + 50) // 100

    @property
    def record_elems(self) -> int:
        return 3 * self.d_model

    @property
    def record_bytes(self) -> int:
        return 3 * self.d_model * 2

    def with_(self, **kw) -> "StackConfig":
        return dataclasses.replace(self, **kw)


# rho of the 7B-class shapes is the value at which this generator gives ~83 %
# token-to-token overlap of the top-k sets (measured by the bench and printed).
CONFIGS = {
    "tiny": StackConfig("tiny", 2, 256, 1024, 64, 10, 20, 16, 0, 0.9),
    "small": StackConfig("small", 3, 512, 2048 + 32, 96, 10, 25, 12, 7, 0.95),
    "7b": StackConfig("7b", 32, 4096, 11008, 512, 10, 25, 128, 1, 0.97),
    "13b": StackConfig("13b", 40, 5120, 13824, 640, 8, 25, 256, 2, 0.97),
    "70b": StackConfig("70b", 80, 8192, 28672, 1024, 5, 20, 128, 3, 0.97),
    "stress": StackConfig("stress", 32, 4096, 11008, 512, 10, 25, 512, 4, 0.97),
}


def _gen(seed: int, tensor_id: int, device: str) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed * _SEED_MUL + tensor_id)
    return g


def _randn_bf16(shape, seed: int, tensor_id: int, device: str, out: Optional[torch.Tensor] = None,
                chunk_elems: int = 1 << 26) -> torch.Tensor:
    """``randn * 0.02`` rounded to bf16, drawn in bounded chunks from one generator."""
    n = math.prod(shape)
    g = _gen(seed, tensor_id, device)
    if out is None:
        out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    assert flat.numel() == n
    for lo in range(0, n, chunk_elems):
        hi = min(n, lo + chunk_elems)
        blk = torch.randn(hi - lo, generator=g, device=device, dtype=torch.float32)
        flat[lo:hi].copy_(blk.mul_(0.02).to(torch.bfloat16))
    return out


def predictor_weights(cfg: StackConfig, device: str = "cpu"):
    """W1 ``[H, D]`` and W2 ``[L*M, H]`` (row-major, layer-major), bf16."""
    w1 = _randn_bf16((cfg.d_pred, cfg.d_model), cfg.seed, 0, device)
    w2 = _randn_bf16((cfg.n_layers * cfg.d_ffn, cfg.d_pred), cfg.seed, 1, device)
    return w1, w2


def fill_backing_store(cfg: StackConfig, out: torch.Tensor, gen_device: str = "cpu") -> torch.Tensor:
    """Fill ``out`` (bf16 ``[L, M, 3, D]``, usually pinned host memory) layer by layer.

    ``gen_device`` may be ``"cuda"`` to draw the large stores quickly; the bytes
    then come from the CUDA generator stream of the same seeds and are copied
    into ``out``.
    """
    L, M, D = cfg.n_layers, cfg.d_ffn, cfg.d_model
    assert tuple(out.shape) == (L, M, 3, D) and out.dtype == torch.bfloat16
    for l in range(L):
        if gen_device == "cpu" and out.device.type == "cpu":
            _randn_bf16((M, 3, D), cfg.seed, 2 + l, "cpu", out=out[l])
        else:
            blk = _randn_bf16((M, 3, D), cfg.seed, 2 + l, gen_device)
            out[l].copy_(blk)
    return out


def backing_store(cfg: StackConfig, pin: bool = False, gen_device: str = "cpu") -> torch.Tensor:
    out = torch.empty((cfg.n_layers, cfg.d_ffn, 3, cfg.d_model), dtype=torch.bfloat16,
                      pin_memory=pin)
    return fill_backing_store(cfg, out, gen_device)


def hidden_states(cfg: StackConfig, n_tokens: Optional[int] = None, batch: int = 1,
                  rho: Optional[float] = None, gamma: float = 0.9) -> torch.Tensor:
    """AR(1) layer-0 hidden states, bf16 ``[T, B, D]`` (CPU generator, fp32 recursion)."""
    T = cfg.n_tokens if n_tokens is None else n_tokens
    rho = cfg.rho if rho is None else rho
    D = cfg.d_model
    g = _gen(cfg.seed, 999, "cpu")
    nproc = 1 if batch == 1 else batch + 1   # [shared driver] + one per sequence
    innov = math.sqrt(max(0.0, 1.0 - rho * rho))
    state = torch.randn(nproc, D, generator=g, dtype=torch.float32)
    out = torch.empty(T, batch, D, dtype=torch.bfloat16)
    for t in range(T):
        if t > 0:
            eps = torch.randn(nproc, D, generator=g, dtype=torch.float32)
            state = rho * state + innov * eps
        if batch == 1:
            out[t, 0] = state[0].to(torch.bfloat16)
        else:
            mix = math.sqrt(gamma) * state[0:1] + math.sqrt(1.0 - gamma) * state[1:]
            out[t] = mix.to(torch.bfloat16)
    return out


def random_bitmaps(n_layers: int, d_ffn: int, n_set: int, seed: int, n_steps: int,
                   persistence: float = 0.8) -> torch.Tensor:
    """Sequence of random predicted bitmaps, int32-typed uint32 words ``[T, L, M/32]``.

    Each step keeps about ``persistence`` of the previous set and redraws the
    rest uniformly; used to drive the residency manager without a predictor.
    Bit ``j`` of word ``w`` stands for neuron ``32 * w + j``.
    """
    assert d_ffn % 32 == 0
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * _SEED_MUL + 31337)
    W = d_ffn // 32
    out = torch.zeros(n_steps, n_layers, W, dtype=torch.int64)
    weights = (1 << torch.arange(32, dtype=torch.int64))
    for l in range(n_layers):
        cur = torch.randperm(d_ffn, generator=g)[:n_set]
        for t in range(n_steps):
            if t > 0:
                keep_n = int(round(persistence * n_set))
                keep = cur[torch.randperm(cur.numel(), generator=g)[:keep_n]]
                mask = torch.ones(d_ffn, dtype=torch.bool)
                mask[cur] = False
                pool = mask.nonzero().flatten()
                new = pool[torch.randperm(pool.numel(), generator=g)[: n_set - keep_n]]
                cur = torch.cat([keep, new])
            bits = torch.zeros(d_ffn, dtype=torch.int64)
            bits[cur] = 1
            out[t, l] = (bits.view(W, 32) * weights).sum(dim=1)
    # store as the uint32 bit pattern inside int32
    out = torch.where(out >= (1 << 31), out - (1 << 32), out)
    return out.to(torch.int32)


def centroid_head_weights(cfg: StackConfig, n_centroids: int, device: str = "cpu") -> torch.Tensor:
    """Head weights of the centroid selection stage, bf16 ``[L * 2 * K, H]``: for each layer the
    K rows of the gate head, then the K rows of the up head (same draw recipe as the other
    predictor weights)."""
    return _randn_bf16((cfg.n_layers * 2 * n_centroids, cfg.d_pred), cfg.seed, 2, device)


def centroid_bank(cfg: StackConfig, n_centroids: int, mask_rows: Optional[int] = None,
                  layers: Optional[int] = None) -> torch.Tensor:
    """A synthetic centroid bank, int32-typed uint32 words ``[L, 2, K, M/32]``.

    Stands in for the bank the method builds offline by clustering thresholded activation masks
    (no trained model is available here).  Every layer has one popularity score per neuron (hot
    neurons recur across centroids, as clustered masks do); centroid ``c`` of head ``h`` is the
    ``mask_rows`` neurons with the highest ``popularity + noise[h, c]``, so every mask has exactly
    the target size, gate and up masks of a layer overlap well above chance, and their
    intersection has a size that varies from pair to pair and never exceeds the mask size.
    ``mask_rows`` defaults to ``top_k``, the target sparsity every centroid is pruned to.  Bit
    ``j`` of word ``w`` stands for neuron ``32 * w + j``.
    """
    L = cfg.n_layers if layers is None else layers
    M, K = cfg.d_ffn, n_centroids
    assert M % 32 == 0
    n_mask = cfg.top_k if mask_rows is None else mask_rows
    g = torch.Generator(device="cpu")
    g.manual_seed(cfg.seed * _SEED_MUL + 4242)
    weights = (1 << torch.arange(32, dtype=torch.int64))
    out = torch.empty((L, 2, K, M // 32), dtype=torch.int32)
    for l in range(L):
        pop = torch.randn(M, generator=g)
        for h in range(2):
            score = pop[None, :] + torch.randn(K, M, generator=g)
            idx = score.topk(n_mask, dim=1).indices
            bits = torch.zeros((K, M), dtype=torch.int64)
            bits.scatter_(1, idx, 1)
            words = (bits.view(K, M // 32, 32) * weights).sum(dim=2)          # < 2**32
            out[l, h] = torch.where(words >= (1 << 31), words - (1 << 32), words).to(torch.int32)
    return out


def quantize_store(store: torch.Tensor, device: str = "cpu", out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """An 8-bit record store made from a bf16 one, uint8 ``[L, M, 3*D + 16]``: per row the int8
    values ``round(w / s)`` with ``s = max|w| / 127`` (fp32; 1 for an all-zero row), then the three
    scales as fp32 and four bytes of padding.  Input preparation only: what a weight *is* after
    this (the product that is rounded back to bf16) is defined by whoever reads the store.
    ``device`` is where the arithmetic runs (layer by layer); the result is a host tensor."""
    L, M, three, D = store.shape
    assert three == 3 and D % 16 == 0
    if out is None:
        out = torch.zeros((L, M, 3 * D + 16), dtype=torch.uint8)
    for l in range(L):
        w = store[l].to(device).to(torch.float32)                        # [M, 3, D]
        s = w.abs().amax(dim=2) / 127.0
        s = torch.where(s > 0, s, torch.ones_like(s))
        q = torch.clamp(torch.round(w / s[..., None]), -127, 127).to(torch.int8)
        rec = torch.zeros((M, 3 * D + 16), dtype=torch.uint8, device=w.device)
        rec[:, :3 * D] = q.reshape(M, 3 * D).view(torch.uint8)
        rec[:, 3 * D:3 * D + 12] = s.contiguous().view(torch.uint8).reshape(M, 12)
        out[l].copy_(rec)
    return out


def trunk_weights(T: int, feature_dims, K0: int, E: int, n_blocks: int, n_heads: int, K: int, seed: int,
                  device: str = "cpu") -> dict:
    """Random weights of the Section 3.3 predictor (projection blocks, centroid embedding, residual
    trunk, centroid heads); stands in for the trained predictor, which is not available.

    Matrices are bf16, row-major ``[out][in]``; biases and LayerNorm gains / biases are fp32.  A
    feature whose dimension is not a multiple of 8 (the scalar norm feature) gets its weight rows
    padded with zero columns to the next multiple of 8, and is passed padded with zeros: the
    products are unchanged.  ``feature_dims`` are the true dimensions.
    """
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * _SEED_MUL + 777)

    def mat(rows, cols, pad_to=None, scale=None):
        scale = (1.0 / max(cols, 1)) ** 0.5 if scale is None else scale
        w = torch.randn(rows, cols, generator=g) * scale
        if pad_to is not None and pad_to != cols:
            w = torch.cat([w, torch.zeros(rows, pad_to - cols)], dim=1)
        return w.to(torch.bfloat16).contiguous().to(device)

    def vec(n, centre=0.0, scale=0.1):
        return (centre + scale * torch.randn(n, generator=g)).to(torch.float32).contiguous().to(device)

    def block(rows, cols, pad_to=None):
        return (mat(rows, cols, pad_to), vec(rows), vec(rows, 1.0), vec(rows))

    w = {"T": T, "K": K, "K0": K0, "E": E, "feature_dims": tuple(feature_dims)}
    w["proj"] = [block(T, d, (d + 7) // 8 * 8) for d in feature_dims]
    w["emb"] = mat(K0, E, scale=1.0)
    w["cproj"] = block(4 * T, E)
    w["blocks"] = []
    for _ in range(n_blocks):
        w1, b1, gain, bias = block(4 * T, 8 * T)
        w["blocks"].append((w1, b1, gain, bias, mat(8 * T, 4 * T), vec(8 * T)))
    w["heads"] = mat(n_heads * 2 * K, 8 * T)
    return w


def trunk_features(feature_dims, n_tokens: int, K0: int, seed: int):
    """Synthetic layer-0 features for ``n_tokens`` tokens: one fp32 ``[n_tokens, pad8(d)]`` tensor
    per continuous feature (zero beyond the true dimension) and int32 centroid IDs ``[n_tokens]``.
    Stand-ins for the embedding, the pre-attention norm output, the attention sketch and the
    post-attention norm of a real model's layer 0."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * _SEED_MUL + 778)
    feats = []
    for d in feature_dims:
        f = torch.zeros(n_tokens, (d + 7) // 8 * 8)
        f[:, :d] = torch.randn(n_tokens, d, generator=g)
        feats.append(f.contiguous())
    ids = torch.randint(0, K0, (n_tokens,), generator=g, dtype=torch.int32)
    return feats, ids
