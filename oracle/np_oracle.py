"""CPU oracle for the delta-prefetch decode hot path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 restatement of what one decode step computes, written from
the paper (Sections 3.1, 3.4, 3.5) and from the workload definition, for the
sole purpose of checking the CUDA library.  It shares no code with that library
and imports nothing from it; only tests, the smoke check and the benchmark's
CPU-baseline leg may import this file.  It is not tuned for speed.

Conventions (same symbols as the C header):
  L layers, D model width, M FFN width (multiple of 32), H predictor width,
  k rows selected per layer per sequence, C resident capacity in rows,
  W = M / 32 bitmap words per layer; bit j of word w is neuron 32*w + j.
  bf16 tensors are passed as ``uint16`` bit patterns.

Pins (see tests/test_oracle_*.py): exact rational brute force and structured
closed forms for ``predict``; full-sort brute force, constructed ties and
degenerate k for ``topk_bitmap``; a per-bit scalar loop, constructed ties and
the one-hot/identity-bank special cases for ``centroid_select``; the set identities of Eq. 2-3, slot-map
bijection invariants and a set-based brute force for ``Residency.delta``
(``validity_errors`` is the order-free form of those invariants, itself checked
on hand-made valid and invalid states);
byte identity for ``install``; the dense SwiGLU library form when every row is
active, linearity over disjoint sets and a scalar loop for ``sparse_mlp``; the
paper's buffer-size arithmetic (Section 4.3) for ``record_bytes``; unit output
RMS, scale invariance and a hand value for ``rms_normalize``; a scan, boundary
budgets and monotonicity for ``dense_prefix_plan``; the dense stack in a
library's fp64 ops and "a dense layer is a sparse layer with every row active"
for the dense prefix of ``Engine``; a library's fp32 -> bf16 conversion (with
constructed ties) and hand values for ``dequantize_records``; the paper's
parameter table for ``trunk_param_counts``, a library's LayerNorm and SiLU for
``layer_norm`` / ``silu``, a scalar restatement on tiny sizes and structural
properties (coordinate-copying heads, vanishing second matrices, the centroid
half of the concatenation) for ``trunk_forward`` (Section 3.3).

``Residency.speculate`` (the deeper prefetch the paper names as future work): it never evicts, keeps
every table valid, leaves the chain's output bit-identical, and under exact replacement the next
step's incoming set shrinks by exactly the speculative rows that are predicted (set brute force).

Parity unpinned against the paper (the paper is silent; these are this build's
definitions, pinned only by invariants and determinism): the candidate and slot rule of
``Residency.speculate``, the victim order of
the LRU policy, the truncation rule when a predicted set exceeds capacity, and
``dense_prefix_plan`` against the paper's own operating points (found there by
a throughput sweep on its device, not by a formula), and the 8-bit record
format of ``dequantize_records`` (the paper names quantised records only as
future work; the rounding itself is pinned against a library conversion).
In ``trunk_forward`` the paper leaves open the LayerNorm epsilon (1e-5 here),
the width of the centroid embedding (2048 reproduces its row of the parameter
table), the shape of the "small projection network" behind it (one block of
the same form as the feature blocks) and whether the heads have biases (none
here; the table's head row is met to 0.14 % either way).
"""
from __future__ import annotations

import numpy as np

EVICT_EXACT = 0   # Eq. 3: every row that leaves the predicted set frees its slot
EVICT_LRU = 1     # keep rows while capacity allows; evict least recently predicted


# --------------------------------------------------------------------------
# layout arithmetic (Section 3.5: neuron-centric records; Section 4.3: sizes)
# --------------------------------------------------------------------------
def record_bytes(D: int, elem_bytes: int = 2) -> int:
    """One neuron record = its gate, up and transposed-down rows, back to back."""
    return 3 * D * elem_bytes


def resident_buffer_bytes(C: int, D: int, elem_bytes: int = 2) -> int:
    """Bytes of one layer's resident row buffers (three projections, C rows each)."""
    return C * record_bytes(D, elem_bytes)


def dense_prefix_plan(L: int, M: int, D: int, C: int, budget_bytes: int, fixed_bytes: int = 0,
                      elem_bytes: int = 2) -> int:
    """Largest dense prefix d (Section 3.1: "the largest dense prefix that fits within the
    memory budget"): d dense layers hold all M records, the other L - d layers a resident
    buffer of C records each, next to ``fixed_bytes`` of other resident state.  Returns -1 when
    not even d = 0 fits.  (The paper finds its operating point by a throughput sweep on its
    device; this is the memory rule that sweep is described by.)"""
    rec = record_bytes(D, elem_bytes)
    best = -1
    for d in range(L + 1):
        if d * M * rec + (L - d) * C * rec + fixed_bytes <= budget_bytes:
            best = d
    return best


def quantized_record_bytes(D: int) -> int:
    """Size of an 8-bit record (a transfer-path variant the paper leaves as future work,
    Section 6): the gate, up and transposed-down rows as int8, D values each, then their three
    fp32 scales and four bytes of padding, so that records stay 16-byte aligned."""
    return 3 * D + 16


def dequantize_records(q_u8: np.ndarray, D: int) -> np.ndarray:
    """8-bit records ``[..., 3*D + 16]`` (uint8) -> bf16 bit patterns ``[..., 3, D]`` (uint16).

    Row p of a record is ``int8 q[p*D:(p+1)*D]`` with scale ``s_p`` (fp32, little endian, at byte
    ``3*D + 4*p``); a weight is ``float32(q) * s_p`` (one fp32 multiplication) rounded to bf16,
    ties to even.  This is this build's definition: the paper does not specify one."""
    q_u8 = np.ascontiguousarray(q_u8, dtype=np.uint8)
    lead = q_u8.shape[:-1]
    assert q_u8.shape[-1] == quantized_record_bytes(D)
    q = q_u8[..., :3 * D].view(np.int8).reshape(*lead, 3, D).astype(np.float32)
    scales = np.ascontiguousarray(q_u8[..., 3 * D:3 * D + 12]).view(np.float32).reshape(*lead, 3)
    w = (q * scales[..., None]).astype(np.float32)          # fp32 product, rounded once
    bits = np.ascontiguousarray(w).view(np.uint32)
    rounded = bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def record_offset_bytes(layer: int, neuron: int, M: int, D: int) -> int:
    """Byte offset of a record in the layer-major store: consecutive neuron IDs
    of a layer occupy consecutive byte ranges (Section 3.5)."""
    return (layer * M + neuron) * record_bytes(D)


def count_from_percent(pct: int, M: int) -> int:
    """Rows for a density or capacity given in percent of M (rounded to nearest)."""
    return (pct * M + 50) // 100


# --------------------------------------------------------------------------
# number formats
# --------------------------------------------------------------------------
def bf16_to_f64(u16: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp64."""
    u16 = np.ascontiguousarray(u16, dtype=np.uint16)
    return (u16.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def fp32_order_key(z32: np.ndarray) -> np.ndarray:
    """Order-preserving map from fp32 bit patterns to uint32 (larger float ->
    larger key; +0 above -0): flip all bits of negatives, set the sign bit of
    the rest."""
    b = np.ascontiguousarray(z32, dtype=np.float32).view(np.uint32)
    neg = (b >> np.uint32(31)).astype(bool)
    return np.where(neg, ~b, b | np.uint32(0x80000000)).astype(np.uint32)


def bitmap_to_bool(words: np.ndarray, M: int) -> np.ndarray:
    """uint32 words ``[..., W]`` -> bool ``[..., M]``."""
    words = np.ascontiguousarray(words).view(np.uint32)
    shifts = np.arange(32, dtype=np.uint32)
    bits = (words[..., :, None] >> shifts) & np.uint32(1)
    return bits.reshape(*words.shape[:-1], words.shape[-1] * 32)[..., :M].astype(bool)


def bool_to_bitmap(bits: np.ndarray) -> np.ndarray:
    """bool ``[..., M]`` (M multiple of 32) -> uint32 words ``[..., M/32]``."""
    bits = np.asarray(bits, dtype=bool)
    M = bits.shape[-1]
    assert M % 32 == 0
    b = bits.reshape(*bits.shape[:-1], M // 32, 32).astype(np.uint64)
    weights = (np.uint64(1) << np.arange(32, dtype=np.uint64))
    return (b * weights).sum(axis=-1).astype(np.uint32)


# --------------------------------------------------------------------------
# stage 1: predictor forward (one pass after layer 0 scores every FFN neuron of
# every downstream layer; Section 3.1 step 2, in the workload's MLP form
# D -> H (ReLU) -> L*M, no biases)
# --------------------------------------------------------------------------
def predict(w1_u16: np.ndarray, w2_u16: np.ndarray, x_u16: np.ndarray, L: int, M: int) -> np.ndarray:
    """logits[b, l, n] = sum_m W2[l*M + n, m] * max(0, sum_j W1[m, j] * x[b, j]), fp64.

    The hidden vector is kept in fp64 (never rounded)."""
    W1 = bf16_to_f64(w1_u16)                       # [H, D]
    x = bf16_to_f64(x_u16)                         # [B, D]
    h = np.maximum(0.0, x @ W1.T)                  # [B, H]
    B = x.shape[0]
    z = np.empty((B, L, M), dtype=np.float64)
    for l in range(L):                             # layer by layer only to bound memory
        W2l = bf16_to_f64(w2_u16[l * M:(l + 1) * M])   # [M, H]
        z[:, l, :] = h @ W2l.T
    return z


# --------------------------------------------------------------------------
# stage 2: per-layer top-k -> active bitmaps (replaces the paper's centroid
# lookup by a fixed budget of k rows per layer, Section 4.1's K_max budgets)
# --------------------------------------------------------------------------
def topk_bitmap(logits_f32: np.ndarray, k: int) -> np.ndarray:
    """For every (sequence, layer): the k largest logits under the total order
    (fp32 key descending, neuron index ascending); OR over sequences.

    ``logits_f32`` is ``[B, L, M]`` float32; returns uint32 ``[L, M/32]``."""
    z = np.ascontiguousarray(logits_f32, dtype=np.float32)
    B, L, M = z.shape
    bits = np.zeros((L, M), dtype=bool)
    for b in range(B):
        for l in range(L):
            key = fp32_order_key(z[b, l]).astype(np.int64)
            order = np.argsort(-key, kind="stable")     # ties keep ascending index
            bits[l, order[:k]] = True
    return bool_to_bitmap(bits)


def centroid_select(logits_f32: np.ndarray, bank_words: np.ndarray):
    """Selection through centroid heads (Section 3.3, third stage of the
    predictor; Section 3.4: the active set is the intersection of the gate and
    the up centroid masks).

    ``logits_f32`` is ``[B, L, 2, K]`` float32: for every sequence and layer
    one row of logits over the centroid vocabulary for the gate head (index 0)
    and one for the up head (index 1).  Each head takes its arg-max centroid
    (ties: the lower centroid ID; order = the fp32 total order used by
    ``topk_bitmap``).  ``bank_words`` is the bit-packed centroid bank
    ``[L, 2, K, W]`` uint32.  The layer's active set for one sequence is
    gate_mask AND up_mask; sequences are ORed.

    Returns ``(ids, words)``: int32 ``[B, L, 2]`` chosen centroid IDs and the
    uint32 bitmap ``[L, W]``."""
    z = np.ascontiguousarray(logits_f32, dtype=np.float32)
    bank = np.ascontiguousarray(bank_words).view(np.uint32)
    B, L, two, K = z.shape
    assert two == 2 and bank.shape[:3] == (L, 2, K)
    W = bank.shape[3]
    ids = np.zeros((B, L, 2), dtype=np.int32)
    words = np.zeros((L, W), dtype=np.uint32)
    for b in range(B):
        for l in range(L):
            for h in range(2):
                key = fp32_order_key(z[b, l, h]).astype(np.int64)
                ids[b, l, h] = int(np.argmax(key))      # first maximum = lowest ID
            words[l] |= bank[l, 0, ids[b, l, 0]] & bank[l, 1, ids[b, l, 1]]
    return ids, words


# --------------------------------------------------------------------------
# the shared predictor of Section 3.3 (features -> projection blocks ->
# residual trunk -> centroid heads), inference only (no dropout)
# --------------------------------------------------------------------------
LN_EPS = 1e-5   # the paper does not state the epsilon of its LayerNorms; the common default is taken


def layer_norm(v: np.ndarray, gain: np.ndarray, bias: np.ndarray) -> np.ndarray:
    """LayerNorm over the last axis: (v - mean) / sqrt(var + eps) * gain + bias, biased variance."""
    v = np.asarray(v, dtype=np.float64)
    mu = v.mean(axis=-1, keepdims=True)
    var = ((v - mu) ** 2).mean(axis=-1, keepdims=True)
    return (v - mu) / np.sqrt(var + LN_EPS) * gain + bias


def silu(v: np.ndarray) -> np.ndarray:
    v = np.asarray(v, dtype=np.float64)
    return v / (1.0 + np.exp(-v))


def trunk_param_counts(T: int, feature_dims, K: int, E: int, n_blocks: int, n_heads: int) -> dict:
    """Parameters per component of the Section 3.3 predictor (the rows of the paper's cost table),
    with a bias on every linear layer but the heads and gain + bias on every LayerNorm."""
    proj = sum(d * T + T + 2 * T for d in feature_dims)
    emb = K * E + (E * 4 * T + 4 * T + 2 * 4 * T)
    trunk = n_blocks * ((8 * T) * (4 * T) + 4 * T + 2 * 4 * T + (4 * T) * (8 * T) + 8 * T)
    heads = 2 * n_heads * K * (8 * T)
    return {"input_projections": proj, "centroid_embedding": emb, "residual_trunk": trunk, "output_heads": heads,
            "total": proj + emb + trunk + heads}


def trunk_forward(w: dict, features, centroid_id: int) -> np.ndarray:
    """Head logits ``[n_heads, 2, K]`` of the Section 3.3 predictor for one token.

    ``features``: the four continuous layer-0 features (vectors of the dims the weights were
    made for).  Stage 1: every feature goes through its own block Linear -> LayerNorm -> SiLU to
    T dims; the layer-0 gate centroid ID goes through an embedding and one such block to 4T dims;
    the five results are concatenated to 8T.  Stage 2: residual blocks
    z <- z + W2 SiLU(LayerNorm(W1 z + b1)) + b2 with W1: 8T -> 4T, W2: 4T -> 8T.  Stage 3: the
    gate head and the up head of every sparse layer, linear, K logits each.
    ``w`` holds fp64 arrays (bf16 values widened by the caller): ``proj[i] = (W, b, gain, bias)``,
    ``emb`` ``[K0, E]``, ``cproj = (W, b, gain, bias)``, ``blocks[j] = (W1, b1, gain, bias, W2, b2)``,
    ``heads`` ``[n_heads * 2 * K, 8T]`` (layer-major, gate head before up head), ``K``.
    """
    parts = []
    for (W, b, g, be), f in zip(w["proj"], features):
        parts.append(silu(layer_norm(W @ np.asarray(f, dtype=np.float64) + b, g, be)))
    W, b, g, be = w["cproj"]
    parts.append(silu(layer_norm(W @ w["emb"][centroid_id] + b, g, be)))
    z = np.concatenate(parts)
    for (W1, b1, g, be, W2, b2) in w["blocks"]:
        z = z + W2 @ silu(layer_norm(W1 @ z + b1, g, be)) + b2
    return (w["heads"] @ z).reshape(-1, 2, w["K"])



# --------------------------------------------------------------------------
# stage 3a: delta / residency (Section 3.4, Eq. 2-3, slot map S in Z^M)
# --------------------------------------------------------------------------
class LayerDelta:
    """What one layer's delta step emits (all ascending neuron index)."""

    def __init__(self):
        self.delta_ids = np.zeros(0, np.int32)     # incoming rows that got a slot
        self.delta_slots = np.zeros(0, np.int32)   # their slots
        self.evict_ids = np.zeros(0, np.int32)     # rows that released their slot
        self.overflow_ids = np.zeros(0, np.int32)  # incoming rows left non-resident
        self.active_ids = np.zeros(0, np.int32)    # predicted AND resident, after update
        self.active_slots = np.zeros(0, np.int32)
        self.n_pred = 0
        self.n_kept = 0


class Residency:
    """Per-layer resident-row state: bitmap R, slot map S (-1 = not resident),
    owner (slot -> neuron, -1 = free) and last-predicted step stamps."""

    def __init__(self, L: int, M: int, C: int, policy: int = EVICT_EXACT):
        assert M % 32 == 0 and 0 < C <= M
        self.L, self.M, self.C, self.policy = L, M, C, policy
        self.reset()

    def reset(self):
        L, M, C = self.L, self.M, self.C
        self.R = np.zeros((L, M), dtype=bool)
        self.S = np.full((L, M), -1, dtype=np.int32)
        self.owner = np.full((L, C), -1, dtype=np.int32)
        self.stamp = np.full((L, M), -1, dtype=np.int32)
        self.t = 0

    def delta(self, pred_words: np.ndarray) -> list:
        """One decode step for all layers.  ``pred_words`` uint32 ``[L, W]``."""
        P_all = bitmap_to_bool(pred_words, self.M)
        out = [self._delta_layer(l, P_all[l]) for l in range(self.L)]
        self.t += 1
        return out

    def _delta_layer(self, l: int, P: np.ndarray) -> LayerDelta:
        R, S, owner, stamp = self.R[l], self.S[l], self.owner[l], self.stamp[l]
        C = self.C
        res = LayerDelta()
        # 1. kept rows, incoming rows (Eq. 2) and eviction candidates (Eq. 3's set)
        kept = np.flatnonzero(P & R)
        D_in = np.flatnonzero(P & ~R)               # ascending neuron index
        cand = np.flatnonzero(R & ~P)
        res.n_pred = int(P.sum())
        res.n_kept = int(kept.size)
        # 2. every predicted row is stamped with the current step
        stamp[P] = self.t
        # 3. victims
        if self.policy == EVICT_EXACT:
            E = cand
        else:
            free = C - int(R.sum())
            need = max(0, int(D_in.size) - free)
            if need >= cand.size:
                E = cand
            else:
                # least recently predicted first, ties by lower neuron index
                order = np.lexsort((cand, stamp[cand]))
                E = np.sort(cand[order[:need]])
        # 4. outgoing rows release their slots
        for n in E:
            owner[S[n]] = -1
            S[n] = -1
            R[n] = False
        res.evict_ids = E.astype(np.int32)
        # 5. i-th incoming row (ascending neuron) takes the i-th free slot (ascending slot)
        avail = np.flatnonzero(owner == -1)
        n_fit = min(int(D_in.size), int(avail.size))
        for i in range(n_fit):
            n, s = int(D_in[i]), int(avail[i])
            S[n] = s
            owner[s] = n
            R[n] = True
        res.delta_ids = D_in[:n_fit].astype(np.int32)
        res.delta_slots = avail[:n_fit].astype(np.int32)
        res.overflow_ids = D_in[n_fit:].astype(np.int32)
        # 6. the rows the sparse MLP will use: predicted and resident
        act = np.flatnonzero(P & R)
        res.active_ids = act.astype(np.int32)
        res.active_slots = S[act].astype(np.int32)
        return res

    def resident_words(self) -> np.ndarray:
        return bool_to_bitmap(self.R)

    def speculate(self, cand_words: np.ndarray, budget: int) -> list:
        """Speculative residency, after this step's ``delta`` and before the next one.

        The paper names a deeper prefetch pipeline as future work (Section 6): rows are fetched
        before a token asks for them.  Residency is a cache (a resident row that is not
        predicted is simply not used), so rows may be made resident ahead of time without
        changing any result; what changes is the next token's incoming set, ``P \\ R``.
        Rule (this build's; the paper gives none): per layer, of the candidate rows that are not
        resident, the ``min(budget, free slots)`` lowest-indexed ones become resident; the i-th
        of them (ascending neuron) takes the i-th free slot (ascending slot), exactly as
        incoming rows do.  Nothing is evicted and no stamp changes, so under the LRU policy a
        speculative row that is never predicted is among the first to leave, and under Eq. 3's
        exact replacement it leaves at the next step.  Returns one ``(ids, slots)`` pair of
        int32 arrays per layer."""
        cand_all = bitmap_to_bool(cand_words, self.M)
        out = []
        for l in range(self.L):
            R, S, owner = self.R[l], self.S[l], self.owner[l]
            want = np.flatnonzero(cand_all[l] & ~R)
            avail = np.flatnonzero(owner == -1)
            n = max(0, min(int(budget), int(want.size), int(avail.size)))
            ids, slots = want[:n].astype(np.int32), avail[:n].astype(np.int32)
            for i in range(n):
                S[ids[i]] = slots[i]
                owner[slots[i]] = ids[i]
                R[ids[i]] = True
            out.append((ids, slots))
        return out


def validity_errors(slot_map: np.ndarray, owner: np.ndarray, resident: np.ndarray, C: int,
                    pred: np.ndarray = None, active_ids: np.ndarray = None) -> list:
    """Order-free validity of one layer's residency state (Section 3.4: "correctness depends on
    row presence and slot address", not on which free slot a row took).  Returns the violated
    conditions as text, an empty list for any correct assignment: the slot map restricted to the
    resident rows is injective into [0, C), absent rows map to -1, ``owner`` is its inverse and -1
    elsewhere, and (when given) the active rows are exactly the predicted rows that are resident.
    Used to tell "wrong" from "differently ordered" when a list differs from the canonical one."""
    errs = []
    S = np.asarray(slot_map)
    R = np.asarray(resident, dtype=bool)
    ow = np.asarray(owner)
    if not ((S >= 0) == R).all():
        errs.append("slot map is >= 0 on a row that is not resident, or -1 on one that is")
    slots = S[R]
    if slots.size and (slots.min() < 0 or slots.max() >= C):
        errs.append("a resident row's slot lies outside [0, C)")
    elif np.unique(slots).size != slots.size:
        errs.append("two resident rows share a slot")
    else:
        if slots.size and not (ow[slots] == np.flatnonzero(R)).all():
            errs.append("owner is not the inverse of the slot map")
        free = np.ones(C, dtype=bool)
        free[slots] = False
        if not (ow[free] == -1).all():
            errs.append("a free slot has an owner")
    if int(R.sum()) > C:
        errs.append("more resident rows than capacity")
    if pred is not None and active_ids is not None:
        want = np.flatnonzero(np.asarray(pred, dtype=bool) & R)
        if not np.array_equal(np.sort(np.asarray(active_ids)), want):
            errs.append("the active rows are not the predicted rows that are resident")
    return errs



# --------------------------------------------------------------------------
# stage 3b/3c: install (Section 3.5: interleaved records -> three row buffers)
# --------------------------------------------------------------------------
def coalesce_runs(ids: np.ndarray) -> list:
    """Ascending IDs -> list of (first_id, count) with adjacent IDs merged."""
    runs = []
    for n in np.asarray(ids, dtype=np.int64):
        if runs and runs[-1][0] + runs[-1][1] == n:
            runs[-1][1] += 1
        else:
            runs.append([int(n), 1])
    return [(a, c) for a, c in runs]


def install(backing_u16: np.ndarray, gate: np.ndarray, up: np.ndarray, downT: np.ndarray,
            layer: int, delta_ids: np.ndarray, delta_slots: np.ndarray) -> int:
    """Copy record (layer, n) to slot s of the three buffers for every (n, s).

    ``backing_u16`` is ``[L, M, 3, D]``; the buffers are ``[L, C, D]``.  Returns
    the bytes copied.  Reads go run by run, as the transfer path would issue
    them; the result does not depend on that grouping."""
    pos = 0
    for first, count in coalesce_runs(delta_ids):
        block = backing_u16[layer, first:first + count]      # [count, 3, D]
        for r in range(count):
            s = int(delta_slots[pos])
            gate[layer, s] = block[r, 0]
            up[layer, s] = block[r, 1]
            downT[layer, s] = block[r, 2]
            pos += 1
    assert pos == len(delta_ids)
    return pos * backing_u16.shape[-1] * 3 * 2


# --------------------------------------------------------------------------
# stage 4: sparse SwiGLU MLP through the slot map (Section 3.4)
# --------------------------------------------------------------------------
def sparse_mlp(gate: np.ndarray, up: np.ndarray, downT: np.ndarray, layer: int,
               slots: np.ndarray, x: np.ndarray) -> np.ndarray:
    """y[b] = sum_i silu(g_i) * u_i * downT[s_i], g_i = gate[s_i] . x[b], u_i = up[s_i] . x[b].

    ``slots`` are the buffer slots of the active rows; ``x`` is fp64 ``[B, D]``."""
    slots = np.asarray(slots, dtype=np.int64)
    x = np.asarray(x, dtype=np.float64)
    G = bf16_to_f64(gate[layer, slots])          # [n, D]
    U = bf16_to_f64(up[layer, slots])
    Dn = bf16_to_f64(downT[layer, slots])
    g = x @ G.T                                  # [B, n]
    u = x @ U.T
    a = g / (1.0 + np.exp(-g)) * u
    return a @ Dn                                # [B, D]


def sparse_mlp_from_store(backing_u16: np.ndarray, layer: int, ids: np.ndarray, x: np.ndarray) -> np.ndarray:
    """Same sum, rows taken straight from the record store by neuron ID."""
    ids = np.asarray(ids, dtype=np.int64)
    x = np.asarray(x, dtype=np.float64)
    rec = backing_u16[layer, ids]                # [n, 3, D]
    G, U, Dn = bf16_to_f64(rec[:, 0]), bf16_to_f64(rec[:, 1]), bf16_to_f64(rec[:, 2])
    g = x @ G.T
    u = x @ U.T
    a = g / (1.0 + np.exp(-g)) * u
    return a @ Dn


# --------------------------------------------------------------------------
# one whole decode step of the stack.  The layers form a pre-normalised residual
# chain, x_{l+1} = x_l + MLP_l(rms_normalize(x_l)), as the MLP blocks of the
# paper's models do (their per-layer normalisation parameters stay resident,
# Section 3.1); the gain is 1.  Without the normalisation a chain of random
# N(0, 0.02) SwiGLU layers of width 4096 overflows within a dozen layers.
# --------------------------------------------------------------------------
RMS_EPS = 1e-6


def rms_normalize(x: np.ndarray) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps) along the last axis."""
    x = np.asarray(x, dtype=np.float64)
    return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + RMS_EPS)


class Engine:
    """State carried across decode steps: residency tables and resident buffers."""

    def __init__(self, L, D, M, H, k, C, policy, w1_u16, w2_u16, backing_u16, dense_layers: int = 0):
        """``dense_layers`` = d: the first d layers are dense (Section 3.1): all their rows are
        resident and used, they are never predicted, diffed or installed; their entries of the
        predicted bitmap are empty and their tables stay empty."""
        assert 0 <= dense_layers <= L
        self.L, self.D, self.M, self.H, self.k, self.C = L, D, M, H, k, C
        self.dense_layers = dense_layers
        self.w1, self.w2, self.backing = w1_u16, w2_u16, backing_u16
        self.res = Residency(L, M, C, policy)
        self.gate = np.zeros((L, C, D), dtype=np.uint16)
        self.up = np.zeros((L, C, D), dtype=np.uint16)
        self.downT = np.zeros((L, C, D), dtype=np.uint16)

    def step(self, x_u16: np.ndarray, pred_words: np.ndarray = None, logits_f32: np.ndarray = None,
             spec_extra: int = 0, spec_words: np.ndarray = None):
        """Run predict -> top-k -> delta -> install -> MLP chain for one token.

        ``pred_words`` (or ``logits_f32``) may be supplied to take the selection
        (or the logits) from elsewhere; returns a dict of everything produced.
        ``spec_extra`` > 0 adds the speculative prefetch of ``Residency.speculate`` behind the
        step: the candidates are the rows ranked k+1 .. k+spec_extra by the same order as the
        selection (or ``spec_words``, a candidate bitmap from elsewhere), the budget per layer is
        ``spec_extra``; their records are installed like incoming rows.  The step's own output
        does not depend on it."""
        out = {}
        if pred_words is None:
            if logits_f32 is None:
                z = predict(self.w1, self.w2, x_u16, self.L, self.M)
                out["logits"] = z
                logits_f32 = z.astype(np.float32)
            pred_words = topk_bitmap(logits_f32, self.k)
        if self.dense_layers:
            pred_words = np.array(pred_words, copy=True)
            pred_words[:self.dense_layers] = 0
        out["pred"] = pred_words
        deltas = self.res.delta(pred_words)
        out["deltas"] = deltas
        nbytes = 0
        for l, d in enumerate(deltas):
            nbytes += install(self.backing, self.gate, self.up, self.downT, l, d.delta_ids, d.delta_slots)
        out["installed_bytes"] = nbytes
        x = bf16_to_f64(x_u16)
        ys = []
        xs = [x]
        all_rows = np.arange(self.M)
        for l, d in enumerate(deltas):
            if l < self.dense_layers:
                y = sparse_mlp_from_store(self.backing, l, all_rows, rms_normalize(x))
            else:
                y = sparse_mlp(self.gate, self.up, self.downT, l, d.active_slots, rms_normalize(x))
            ys.append(y)
            x = x + y
            xs.append(x)
        out["y_layers"] = ys
        out["x_layers"] = xs
        out["x_final"] = x
        if spec_extra > 0:
            if spec_words is None:
                assert logits_f32 is not None, "the candidate rule ranks this step's logits"
                spec_words = topk_bitmap(logits_f32, min(self.M, self.k + spec_extra))
            if self.dense_layers:
                spec_words = np.array(spec_words, copy=True)
                spec_words[:self.dense_layers] = 0
            specs = self.res.speculate(spec_words, spec_extra)
            for l, (ids, slots) in enumerate(specs):
                nbytes += install(self.backing, self.gate, self.up, self.downT, l, ids, slots)
            out["specs"] = specs
            out["installed_bytes"] = nbytes
        return out
