"""Thin ctypes binding of ``libnp.so``: argument marshalling only.

Every function has the name and meaning of the C entry point it wraps (see
``include/np.h``).  Tensors are passed as raw pointers; nothing is computed in
Python.  ``Engine`` is a convenience owner of the caller-side buffers (device
memory, pinned host memory and streams come from PyTorch).

There is no fallback: if the compiled library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libnp.so")

NP_OK, NP_E_INVAL, NP_E_STATE, NP_E_CUDA, NP_E_NOMEM, NP_E_DEVICE, NP_E_IO = 0, -1, -2, -3, -4, -5, -6
NP_W_OVERFLOW, NP_W_CHUNKED = 1, 2
NP_EVICT_EXACT, NP_EVICT_LRU = 0, 1
NP_XFER_MEMCPY_RUNS, NP_XFER_HOST_GATHER, NP_XFER_ZERO_COPY, NP_XFER_FILE = 0, 1, 2, 3
NP_F_CHECK_BOUNDS = 1
NP_F_DIRECT_LOADS = 2
NP_F_LAYER_LAUNCHES = 4
NP_F_MAPPED_STAGING = 16
NP_F_NO_TENSOR_CORES = 8
NP_F_ROW_CHAIN = 32
NP_F_CLUSTER_ROWS = 64
NP_F_TCGEN05_BATCH = 128
NP_REC_BF16, NP_REC_INT8 = 0, 1
(NP_CNT_PRED, NP_CNT_KEPT, NP_CNT_DELTA, NP_CNT_EVICT, NP_CNT_OVERFLOW, NP_CNT_ACTIVE,
 NP_CNT_RESIDENT, NP_CNT_STEP) = range(8)
NP_N_COUNTERS = 8

EXPORTED = [
    "np_version", "np_query_sizes", "np_plan_dense_prefix", "np_init", "np_destroy", "np_reset", "np_last_error",
    "np_predict", "np_topk", "np_centroid_select", "np_delta", "np_read_records", "np_install", "np_sparse_mlp", "np_step", "np_step_selected", "np_get_delta",
    "np_read_counters", "np_export_state", "np_import_state", "np_last_step_times", "np_mlp_chain",
    "np_launch_count", "np_chain_launches", "np_speculate", "np_install_speculative", "np_get_speculative", "np_mlp_kernel_name", "np_selftest_bounded_wait", "np_predict_logits_noalloc", "np_noalloc_check", "np_noalloc_last_error",
    "np_trunk_workspace_floats", "np_trunk_forward", "np_trunk_last_error",
]


class np_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "n_layers", "d_model", "d_ffn", "d_pred", "top_k", "capacity", "max_batch", "evict_policy",
        "staging_rows", "transfer_mode", "flags", "host_threads", "chain_layers", "ring_stages",
        "dense_layers", "record_format", "io_depth", "store_layers", "spec_rows", "reserved")]


class np_sizes(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in (
        "w1_bytes", "w2_bytes", "backing_bytes", "row_buffer_bytes", "staging_bytes", "workspace_bytes",
        "host_lists_bytes", "logits_bytes", "bitmap_bytes", "record_bytes", "dense_bytes")]


class np_buffers(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "w1", "w2", "backing", "gate_buf", "up_buf", "downT_buf", "staging", "host_staging", "workspace",
        "host_lists", "dense_buf")] + [("backing_fd", C.c_int32), ("reserved", C.c_int32)]


NP_TRUNK_MAX_BLOCKS = 16


class np_trunk_desc(C.Structure):
    _fields_ = [("T", C.c_int32), ("n_features", C.c_int32), ("feature_dim", C.c_int32 * 4), ("K0", C.c_int32),
                ("E", C.c_int32), ("n_blocks", C.c_int32), ("n_heads", C.c_int32), ("K", C.c_int32),
                ("reserved", C.c_int32 * 5)]


class np_trunk_weights(C.Structure):
    _fields_ = [("proj_w", C.c_void_p * 4), ("proj_b", C.c_void_p * 4), ("proj_gain", C.c_void_p * 4),
                ("proj_bias", C.c_void_p * 4), ("emb", C.c_void_p), ("cproj_w", C.c_void_p), ("cproj_b", C.c_void_p),
                ("cproj_gain", C.c_void_p), ("cproj_bias", C.c_void_p)] + [
        (n, C.c_void_p * NP_TRUNK_MAX_BLOCKS) for n in ("blk_w1", "blk_b1", "blk_gain", "blk_bias", "blk_w2", "blk_b2")
    ] + [("heads", C.c_void_p)]


class np_delta_view(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "delta_ids", "delta_slots", "evict_ids", "overflow_ids", "active_ids", "active_slots", "counters")]


class NpError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"libnp error {code}: {msg}")
        self.code = code


_lib = None


def load() -> C.CDLL:
    """Load ``libnp.so`` (once) and declare the signatures."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2608_22643_b200.build` "
            "(there is no CPU or PyTorch fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, i32 = C.c_void_p, C.c_int32
    lib.np_version.restype = C.c_int
    lib.np_last_error.restype = C.c_char_p
    lib.np_trunk_last_error.restype = C.c_char_p
    lib.np_trunk_last_error.argtypes = []
    lib.np_last_error.argtypes = [vp]
    sigs = {
        "np_query_sizes": [C.POINTER(np_config), C.POINTER(np_sizes)],
        "np_plan_dense_prefix": [C.POINTER(np_config), C.c_uint64, C.c_uint64, C.POINTER(C.c_int32)],
        "np_init": [C.POINTER(vp), C.POINTER(np_config), C.POINTER(np_buffers)],
        "np_destroy": [vp],
        "np_reset": [vp, vp],
        "np_predict": [vp, vp, i32, vp, vp, vp],
        "np_topk": [vp, vp, i32, vp, vp],
        "np_centroid_select": [vp, vp, i32, i32, vp, vp, vp, vp],
        "np_delta": [vp, vp, vp],
        "np_install": [vp, i32, i32, vp],
        "np_trunk_workspace_floats": [C.POINTER(np_trunk_desc), C.POINTER(C.c_uint64)],
        "np_trunk_forward": [C.POINTER(np_trunk_desc), C.POINTER(np_trunk_weights), C.POINTER(vp), vp, vp, vp, vp],
        "np_read_records": [i32, C.c_uint64, C.c_uint64, vp, i32, vp, i32, vp, vp],
        "np_sparse_mlp": [vp, i32, vp, i32, vp, vp],
        "np_step": [vp, vp, i32, vp, vp, vp],
        "np_step_selected": [vp, vp, i32, vp, vp, vp, vp],
        "np_get_delta": [vp, i32, C.POINTER(np_delta_view)],
        "np_read_counters": [vp, vp, vp],
        "np_export_state": [vp, i32, vp, vp, vp, vp, vp],
        "np_import_state": [vp, i32, vp, vp, vp, vp, i32, vp],
        "np_last_step_times": [vp, vp],
        "np_mlp_chain": [vp, vp, i32, vp, vp],
        "np_selftest_bounded_wait": [vp, vp],
        "np_launch_count": [vp, C.POINTER(C.c_uint64)],
    }
    lib.np_mlp_kernel_name.restype = C.c_char_p
    lib.np_mlp_kernel_name.argtypes = [vp, i32]
    lib.np_noalloc_last_error.restype = C.c_char_p
    lib.np_noalloc_last_error.argtypes = []
    sigs["np_predict_logits_noalloc"] = [vp, vp, vp, i32, i32, i32, i32, i32, vp, vp]
    sigs["np_noalloc_check"] = [vp]
    sigs["np_speculate"] = [vp, vp, i32, vp]
    sigs["np_chain_launches"] = [vp, C.POINTER(C.c_int32)]
    sigs["np_install_speculative"] = [vp, vp]
    sigs["np_get_speculative"] = [vp, i32, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp)]
    for name, args in sigs.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = C.c_int
    _lib = lib
    return lib


def _ptr(t) -> Optional[int]:
    """Raw address of a tensor / numpy array / int / None."""
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        assert t.is_contiguous()
        return t.data_ptr()
    if isinstance(t, np.ndarray):
        assert t.flags["C_CONTIGUOUS"]
        return t.ctypes.data
    return int(t)


def _stream(s) -> Optional[int]:
    if s is None:
        return None
    if isinstance(s, torch.cuda.Stream):
        return s.cuda_stream
    return int(s)


def _check(ctx, rc: int) -> int:
    if rc < 0:
        raise NpError(rc, load().np_last_error(ctx).decode())
    return rc


# ---- one Python function per C entry point --------------------------------------------
def np_version() -> int:
    return load().np_version()


def np_last_error(ctx=None) -> str:
    return load().np_last_error(ctx).decode()


def np_query_sizes(cfg: np_config) -> np_sizes:
    out = np_sizes()
    _check(None, load().np_query_sizes(C.byref(cfg), C.byref(out)))
    return out


def np_plan_dense_prefix(cfg: np_config, budget_bytes: int, fixed_bytes: int = 0) -> int:
    """Largest dense prefix that fits the budget (-1: not even none); see include/np.h."""
    out = C.c_int32()
    _check(None, load().np_plan_dense_prefix(C.byref(cfg), budget_bytes, fixed_bytes, C.byref(out)))
    return out.value


def np_init(cfg: np_config, bufs: np_buffers) -> int:
    ctx = C.c_void_p()
    _check(None, load().np_init(C.byref(ctx), C.byref(cfg), C.byref(bufs)))
    return ctx.value


def np_destroy(ctx) -> int:
    return load().np_destroy(ctx)


def np_reset(ctx, stream=None) -> int:
    return _check(ctx, load().np_reset(ctx, _stream(stream)))


def np_predict(ctx, x_bf16, B: int, logits_out=None, bitmap_out=None, stream=None) -> int:
    return _check(ctx, load().np_predict(ctx, _ptr(x_bf16), B, _ptr(logits_out), _ptr(bitmap_out),
                                         _stream(stream)))


def np_topk(ctx, logits, B: int, bitmap_out, stream=None) -> int:
    return _check(ctx, load().np_topk(ctx, _ptr(logits), B, _ptr(bitmap_out), _stream(stream)))


def np_centroid_select(ctx, logits, B: int, K: int, bank, ids_out, bitmap_out, stream=None) -> int:
    return _check(ctx, load().np_centroid_select(ctx, _ptr(logits), B, K, _ptr(bank), _ptr(ids_out),
                                                 _ptr(bitmap_out), _stream(stream)))


def np_delta(ctx, pred_bitmap=None, stream=None) -> int:
    return _check(ctx, load().np_delta(ctx, _ptr(pred_bitmap), _stream(stream)))


def np_read_records(fd: int, base_offset: int, rec_bytes: int, ids: np.ndarray, dst: np.ndarray, io_depth: int = 0):
    """Reads the records ``ids`` (ascending) of a store file into ``dst``; returns
    ``(coalesced ranges, whether io_uring carried the reads)``."""
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    assert dst.flags["C_CONTIGUOUS"] and dst.nbytes >= ids.size * rec_bytes
    ranges, ring = C.c_int32(0), C.c_int32(0)
    rc = load().np_read_records(fd, base_offset, rec_bytes, ids.ctypes.data, ids.size, dst.ctypes.data, io_depth,
                                C.addressof(ranges), C.addressof(ring))
    _check(None, rc)
    return ranges.value, bool(ring.value)


def trunk_pack(w: dict, n_heads: int):
    """The C descriptor and pointer table for a weight dict of ``synth.trunk_weights`` whose tensors
    live on the device (the dict must stay alive while the table is in use)."""
    d = np_trunk_desc()
    d.T, d.n_features, d.K0, d.E, d.K = w["T"], 4, w["K0"], w["E"], w["K"]
    d.n_blocks, d.n_heads = len(w["blocks"]), n_heads
    for i, dim in enumerate(w["feature_dims"]):
        d.feature_dim[i] = (dim + 7) // 8 * 8
    t = np_trunk_weights()
    for i, (W, b, g, be) in enumerate(w["proj"]):
        t.proj_w[i], t.proj_b[i], t.proj_gain[i], t.proj_bias[i] = W.data_ptr(), b.data_ptr(), g.data_ptr(), be.data_ptr()
    t.emb = w["emb"].data_ptr()
    W, b, g, be = w["cproj"]
    t.cproj_w, t.cproj_b, t.cproj_gain, t.cproj_bias = W.data_ptr(), b.data_ptr(), g.data_ptr(), be.data_ptr()
    for j, (W1, b1, g, be, W2, b2) in enumerate(w["blocks"]):
        t.blk_w1[j], t.blk_b1[j], t.blk_gain[j], t.blk_bias[j] = W1.data_ptr(), b1.data_ptr(), g.data_ptr(), be.data_ptr()
        t.blk_w2[j], t.blk_b2[j] = W2.data_ptr(), b2.data_ptr()
    t.heads = w["heads"].data_ptr()
    return d, t


def np_trunk_workspace_floats(desc: np_trunk_desc) -> int:
    out = C.c_uint64(0)
    rc = load().np_trunk_workspace_floats(C.byref(desc), C.byref(out))
    if rc < 0:
        raise NpError(rc, load().np_trunk_last_error().decode())
    return int(out.value)


def np_trunk_forward(desc, table, features, centroid_id, workspace, head_logits, stream=None) -> int:
    """``features``: four device fp32 vectors; ``centroid_id``: device int32 scalar."""
    ptrs = (C.c_void_p * 4)(*[_ptr(f) for f in features])
    rc = load().np_trunk_forward(C.byref(desc), C.byref(table), ptrs, _ptr(centroid_id), _ptr(workspace),
                                 _ptr(head_logits), _stream(stream))
    if rc < 0:
        raise NpError(rc, load().np_trunk_last_error().decode())
    return rc


def np_install(ctx, layer_begin: int, layer_end: int, copy_stream=None) -> int:
    return _check(ctx, load().np_install(ctx, layer_begin, layer_end, _stream(copy_stream)))


def np_sparse_mlp(ctx, layer: int, x, B: int, y, stream=None) -> int:
    return _check(ctx, load().np_sparse_mlp(ctx, layer, _ptr(x), B, _ptr(y), _stream(stream)))


def np_step(ctx, x_bf16, B: int, x_out, stream, copy_stream) -> int:
    return _check(ctx, load().np_step(ctx, _ptr(x_bf16), B, _ptr(x_out), _stream(stream),
                                      _stream(copy_stream)))


def np_step_selected(ctx, x_bf16, B: int, bitmap, x_out, stream=None, copy_stream=None) -> int:
    return _check(ctx, load().np_step_selected(ctx, _ptr(x_bf16), B, _ptr(bitmap), _ptr(x_out), _stream(stream),
                                               _stream(copy_stream)))


def np_get_delta(ctx, layer: int) -> np_delta_view:
    out = np_delta_view()
    _check(ctx, load().np_get_delta(ctx, layer, C.byref(out)))
    return out


def np_read_counters(ctx, out_host: np.ndarray, stream=None) -> int:
    return _check(ctx, load().np_read_counters(ctx, _ptr(out_host), _stream(stream)))


def np_export_state(ctx, layer: int, slot_map=None, owner=None, resident=None, stamp=None, stream=None) -> int:
    return _check(ctx, load().np_export_state(ctx, layer, _ptr(slot_map), _ptr(owner), _ptr(resident),
                                              _ptr(stamp), _stream(stream)))


def np_import_state(ctx, layer: int, slot_map, owner, resident, stamp, step: int, stream=None) -> int:
    return _check(ctx, load().np_import_state(ctx, layer, _ptr(slot_map), _ptr(owner), _ptr(resident),
                                              _ptr(stamp), step, _stream(stream)))


def np_last_step_times(ctx) -> np.ndarray:
    out = np.zeros(4, dtype=np.float32)
    _check(ctx, load().np_last_step_times(ctx, _ptr(out)))
    return out


def np_mlp_chain(ctx, x_bf16, B: int, x_out, stream=None) -> int:
    return _check(ctx, load().np_mlp_chain(ctx, _ptr(x_bf16), B, _ptr(x_out), _stream(stream)))


def np_selftest_bounded_wait(ctx, stream=None) -> int:
    """Returns the raw code (NP_E_DEVICE when the bounded wait timed out as designed)."""
    return load().np_selftest_bounded_wait(ctx, _stream(stream))


def np_launch_count(ctx) -> int:
    out = C.c_uint64()
    _check(ctx, load().np_launch_count(ctx, C.byref(out)))
    return int(out.value)


def np_predict_logits_noalloc(w1, w2, x_bf16, B: int, n_layers: int, d_model: int, d_ffn: int, d_pred: int,
                              logits_out, stream=None) -> int:
    """Predictor logits without a context and without allocating (see include/np.h)."""
    rc = load().np_predict_logits_noalloc(_ptr(w1), _ptr(w2), _ptr(x_bf16), B, n_layers, d_model, d_ffn,
                                          d_pred, _ptr(logits_out), _stream(stream))
    if rc < 0:
        raise NpError(rc, load().np_noalloc_last_error().decode())
    return rc


def np_speculate(ctx, cand_bitmap, budget: int, stream=None) -> int:
    return _check(ctx, load().np_speculate(ctx, _ptr(cand_bitmap), budget, _stream(stream)))


def np_install_speculative(ctx, copy_stream=None) -> int:
    return _check(ctx, load().np_install_speculative(ctx, _stream(copy_stream)))


def np_chain_launches(ctx) -> int:
    out = C.c_int32(0)
    _check(ctx, load().np_chain_launches(ctx, C.byref(out)))
    return int(out.value)


def np_mlp_kernel_name(ctx, B: int = 1) -> str:
    name = load().np_mlp_kernel_name(ctx, B)
    return name.decode() if name else ""


def np_noalloc_check(stream=None) -> int:
    """Waits for `stream`; raises if the last allocation-free predictor call recorded a status bit."""
    rc = load().np_noalloc_check(_stream(stream))
    if rc < 0:
        raise NpError(rc, load().np_noalloc_last_error().decode())
    return rc


# ---- buffer owner ----------------------------------------------------------------------
def make_config(L, D, M, H, k, Cap, max_batch=1, evict_policy=NP_EVICT_EXACT, staging_rows=None,
                transfer_mode=NP_XFER_MEMCPY_RUNS, flags=0, host_threads=0, chain_layers=0, ring_stages=0,
                dense_layers=0, record_format=0, io_depth=0, store_layers=0, spec_rows=0) -> np_config:
    cfg = np_config()
    cfg.n_layers, cfg.d_model, cfg.d_ffn, cfg.d_pred = L, D, M, H
    cfg.top_k, cfg.capacity, cfg.max_batch = k, Cap, max_batch
    cfg.evict_policy, cfg.transfer_mode, cfg.flags, cfg.host_threads = evict_policy, transfer_mode, flags, host_threads
    cfg.chain_layers = chain_layers
    cfg.ring_stages = ring_stages
    cfg.dense_layers = dense_layers
    cfg.record_format = record_format
    cfg.io_depth = io_depth
    cfg.store_layers = store_layers
    cfg.spec_rows = spec_rows
    cfg.staging_rows = staging_rows if staging_rows is not None else max(2, min(Cap, 2 * max(1, k)))
    return cfg


def replica_host_threads(local_world_size: int) -> int:
    """Packing threads for one of ``local_world_size`` contexts that share a host (NP_XFER_HOST_GATHER).

    A context on its own takes all cores but two (``host_threads = 0``); replicas on one host get an equal
    share of that, at least one each, so that N contexts do not start N times the host's cores in threads.
    """
    cores = os.cpu_count() or 1
    return max(1, (cores - 2) // max(1, local_world_size))


def pin_host_tensor(t: torch.Tensor) -> None:
    """Page-lock an existing CPU tensor in place (exact size, no pool rounding)."""
    rc = torch.cuda.cudart().cudaHostRegister(t.data_ptr(), t.numel() * t.element_size(), 0)
    if int(rc) != 0:
        raise RuntimeError(f"cudaHostRegister failed with {rc}")


def unpin_host_tensor(t: torch.Tensor) -> None:
    torch.cuda.cudart().cudaHostUnregister(t.data_ptr())


class _DeviceInts:
    """int32 view of raw device memory, for torch.as_tensor."""

    def __init__(self, addr: int, n: int):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": "<i4", "data": (addr, False), "version": 2}


class Engine:
    """Owns the caller-side buffers of one context and forwards to the C calls.

    ``w1``/``w2`` are bf16 device tensors, ``backing`` a bf16 CPU tensor
    ``[L, M, 3, D]`` (it is page-locked here if it is not already).  With
    ``NP_XFER_FILE`` the store is a file instead: ``backing`` is ``None`` and
    ``store_path`` names it; it is opened with ``O_DIRECT`` when the file
    system allows (``direct_io`` says whether it was)."""

    def __init__(self, cfg: np_config, w1: torch.Tensor, w2: torch.Tensor, backing: Optional[torch.Tensor],
                 device: str = "cuda:0", store_path: Optional[str] = None, direct: bool = True):
        self.cfg = cfg
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.sizes = np_query_sizes(cfg)
        L, D, M, Cap = cfg.n_layers, cfg.d_model, cfg.d_ffn, cfg.capacity
        assert w1.is_cuda and w2.is_cuda
        assert w1.numel() * 2 == self.sizes.w1_bytes and w2.numel() * 2 == self.sizes.w2_bytes
        self.w1, self.w2, self.backing = w1.contiguous(), w2.contiguous(), backing
        self._registered = False
        self.store_fd, self.direct_io = -1, False
        if cfg.transfer_mode == NP_XFER_FILE:
            assert backing is None and store_path is not None
            if direct:
                try:
                    self.store_fd = os.open(store_path, os.O_RDONLY | os.O_DIRECT)
                    self.direct_io = True
                except OSError:
                    self.store_fd = -1
            if self.store_fd < 0:
                self.store_fd = os.open(store_path, os.O_RDONLY)
        else:
            assert not backing.is_cuda
            assert backing.numel() * backing.element_size() == self.sizes.backing_bytes and backing.is_contiguous()
            if not backing.is_pinned():
                pin_host_tensor(backing)
                self._registered = True
        dev = self.device
        nd = cfg.dense_layers                       # leading dense layers: no slot buffers, one record buffer
        self.gate = torch.zeros((L - nd, Cap, D), dtype=torch.bfloat16, device=dev)
        self.up = torch.zeros((L - nd, Cap, D), dtype=torch.bfloat16, device=dev)
        self.downT = torch.zeros((L - nd, Cap, D), dtype=torch.bfloat16, device=dev)
        self.dense = torch.empty((nd, M, 3, D), dtype=torch.bfloat16, device=dev) if nd else None
        self.staging = torch.empty(int(self.sizes.staging_bytes), dtype=torch.uint8, device=dev)
        self.host_staging = None
        self._staging_registered = False
        if cfg.transfer_mode == NP_XFER_HOST_GATHER:
            self.host_staging = torch.empty(int(self.sizes.staging_bytes), dtype=torch.uint8).pin_memory()
        elif cfg.transfer_mode == NP_XFER_FILE:
            # page-aligned (direct reads land here), page-locked in place
            raw = torch.empty(int(self.sizes.staging_bytes) + 4096, dtype=torch.uint8)
            skip = (-raw.data_ptr()) % 4096
            self.host_staging = raw[skip:skip + int(self.sizes.staging_bytes)]
            self._host_staging_raw = raw
            pin_host_tensor(self.host_staging)
            self._staging_registered = True
        self.workspace = torch.empty(int(self.sizes.workspace_bytes) + 256, dtype=torch.uint8, device=dev)
        ws_ptr = (self.workspace.data_ptr() + 255) // 256 * 256
        self.host_lists = torch.zeros(int(self.sizes.host_lists_bytes) // 4, dtype=torch.int32).pin_memory()
        b = np_buffers()
        b.w1, b.w2 = self.w1.data_ptr(), self.w2.data_ptr()
        b.backing = backing.data_ptr() if backing is not None else None
        b.backing_fd = self.store_fd
        if L - nd > 0:
            b.gate_buf, b.up_buf, b.downT_buf = self.gate.data_ptr(), self.up.data_ptr(), self.downT.data_ptr()
        b.staging = self.staging.data_ptr()
        b.host_staging = self.host_staging.data_ptr() if self.host_staging is not None else None
        b.workspace, b.host_lists = ws_ptr, self.host_lists.data_ptr()
        b.dense_buf = self.dense.data_ptr() if self.dense is not None else None
        self.bufs = b
        self.ctx = np_init(cfg, b)
        self.stream = torch.cuda.Stream(device=dev)
        self.copy_stream = torch.cuda.Stream(device=dev)

    def close(self):
        if getattr(self, "ctx", None):
            np_destroy(self.ctx)
            self.ctx = None
        if self._registered:
            unpin_host_tensor(self.backing)
            self._registered = False
        if getattr(self, "_staging_registered", False):
            unpin_host_tensor(self.host_staging)
            self._staging_registered = False
        if getattr(self, "store_fd", -1) >= 0:
            os.close(self.store_fd)
            self.store_fd = -1

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- helpers that read device lists back for tests and reports --
    def counters(self) -> np.ndarray:
        out = np.zeros((self.cfg.n_layers, NP_N_COUNTERS), dtype=np.int32)
        np_read_counters(self.ctx, out, self.stream)
        return out

    def _read_i32(self, addr: int, n: int) -> np.ndarray:
        if n == 0:
            return np.zeros(0, dtype=np.int32)
        return torch.as_tensor(_DeviceInts(addr, n), device=self.device).cpu().numpy()

    def delta_lists(self, layer: int, counters_row: np.ndarray) -> dict:
        self.stream.synchronize()
        v = np_get_delta(self.ctx, layer)
        c = counters_row
        return {
            "delta_ids": self._read_i32(v.delta_ids, int(c[NP_CNT_DELTA])),
            "delta_slots": self._read_i32(v.delta_slots, int(c[NP_CNT_DELTA])),
            "evict_ids": self._read_i32(v.evict_ids, int(c[NP_CNT_EVICT])),
            "overflow_ids": self._read_i32(v.overflow_ids, int(c[NP_CNT_OVERFLOW])),
            "active_ids": self._read_i32(v.active_ids, int(c[NP_CNT_ACTIVE])),
            "active_slots": self._read_i32(v.active_slots, int(c[NP_CNT_ACTIVE])),
        }

    def speculative_lists(self, layer: int):
        """(ids, slots) of the layer's rows made resident by the last np_speculate."""
        torch.cuda.synchronize(self.device)
        ids, slots, cnt = C.c_void_p(), C.c_void_p(), C.c_void_p()
        _check(self.ctx, load().np_get_speculative(self.ctx, layer, C.byref(ids), C.byref(slots), C.byref(cnt)))
        n = int(self._read_i32(cnt.value, 1)[0])
        return self._read_i32(ids.value, n), self._read_i32(slots.value, n)

    def export_state(self, layer: int) -> dict:
        M, Cap, W = self.cfg.d_ffn, self.cfg.capacity, self.cfg.d_ffn // 32
        S = np.empty(M, np.int32)
        owner = np.empty(Cap, np.int32)
        R = np.empty(W, np.uint32)
        stamp = np.empty(M, np.int32)
        np_export_state(self.ctx, layer, S, owner, R, stamp, self.stream)
        return {"slot_map": S, "owner": owner, "resident": R, "stamp": stamp}
