#!/usr/bin/env python
"""Decode-step benchmark of the delta-prefetch sparse-MLP path.

  python bench.py --gpus N --steps K --warmup W            # the CUDA library
  python bench.py --impl reference --steps K --warmup W    # the CPU oracle, as it stands

A step is one pass of the whole hot path (predict -> top-k -> delta -> install ->
sparse MLP chain) over one decode token of the seeded synthetic 7B-shaped stack.
`value` is measured with the token's hidden state already in HBM; `e2e` with the
hidden state in pinned host memory and the result read back every step.  The
record store lives in pinned host memory in both (it stands in for the NVMe
file), so the install traffic crosses PCIe inside every timed step.

With N > 1 (torchrun) every rank runs an independent replica of the stack on
its own sequence: the path has no exchange step, so there is no collective.
Prints exactly one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_22643_b200 import synth  # noqa: E402

METRIC = "decode steps/s (predict+delta+install+sparse MLP, 7B shape)"
UNIT = "steps/s"
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes per layer (dram__bytes_read.sum + dram__bytes_write.sum of one launch / its layers) of the
# sparse-MLP kernels, from the ncu captures summarised under profiles/: (kernel, config) -> (bytes, file)
NCU_TRAFFIC = {
    ("k_mlp_slices", "7b"): (27.201e6, "profiles/k_mlp_slices_7b.md"),
    ("k_mlp_slices", "13b"): (34.084e6, "profiles/k_mlp_slices_13b.md"),
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=120)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--config", default="7b", choices=sorted(synth.CONFIGS))
    ap.add_argument("--policy", default="exact", choices=["exact", "lru"])
    ap.add_argument("--transfer", default="gather", choices=["runs", "gather", "zerocopy", "file"],
                    help="file: the record store is a file, read through io_uring with O_DIRECT (Section 3.5)")
    ap.add_argument("--mapped-staging", action="store_true",
                    help="gather / file transfer: the scatter kernel reads the pinned staging itself, no staging copy")
    ap.add_argument("--store-path", default=None, help="--transfer file: where the store file is written (default: a temp file)")
    ap.add_argument("--io-depth", type=int, default=0, help="--transfer file: reads in flight (0 = 256; -1 = blocking preads)")
    ap.add_argument("--buffered", action="store_true", help="--transfer file: open the store without O_DIRECT")
    ap.add_argument("--rho", type=float, default=None)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-baseline-steps", type=int, default=3)
    ap.add_argument("--layer-launches", action="store_true", help="one MLP kernel launch per layer")
    ap.add_argument("--direct-loads", action="store_true", help="MLP rows by plain global loads")
    ap.add_argument("--chain-layers", type=int, default=0, help="layers per resident MLP kernel")
    ap.add_argument("--mlp-kernel", default="auto", choices=["auto", "cluster-rows", "row-chain"],
                    help="resident sparse-MLP kernel for one sequence: the library's choice, whole rows per block with "
                         "blocks in clusters (NP_F_CLUSTER_ROWS), or whole rows with a global reduction only (NP_F_ROW_CHAIN)")
    ap.add_argument("--batch-up-kernel", default="mma-sync", choices=["mma-sync", "tcgen05"],
                    help="--batch > 1: the up phase of the batched sparse MLP on the mma.sync kernel or the tcgen05 one "
                         "(NP_F_TCGEN05_BATCH)")
    ap.add_argument("--capacity-pct", type=int, default=None, help="resident capacity in percent of FFN rows")
    ap.add_argument("--store-layers", default="auto",
                    help="layers of records the host store holds (layer l reads layer l mod this); 'auto' = all of them "
                         "unless the host cannot hold and pin the whole store, 0 = all")
    ap.add_argument("--spec-rows", type=int, default=0,
                    help="speculative prefetch behind every step: rows ranked k+1 .. k+N of the step's logits per layer")
    ap.add_argument("--min-timed-steps", type=int, default=240,
                    help="the timed region repeats the K steps (the sequence simply continues) until it spans at "
                         "least this many; ms_per_step is the mean over all of them")
    ap.add_argument("--batch", type=int, default=1, help="sequences per step (the metric's workload is 1)")
    ap.add_argument("--gamma", type=float, default=0.9, help="shared-driver weight of batched hidden states")
    ap.add_argument("--host-threads", type=int, default=0, help="threads packing records (gather transfer)")
    ap.add_argument("--dense-layers", type=int, default=0,
                    help="dense prefix: the first d layers stay whole on the GPU and take no part in selection or install")
    ap.add_argument("--budget-gib", type=float, default=None,
                    help="device memory for MLP weights: the dense prefix becomes the longest one that fits (memory rule)")
    ap.add_argument("--records", default="bf16", choices=["bf16", "int8"],
                    help="int8: the store holds 8-bit rows with fp32 scales, dequantised to bf16 at install (a variant)")
    ap.add_argument("--no-variants", action="store_true",
                    help="skip the extra measurement of the zero-copy transfer mode (default run only)")
    ap.add_argument("--selection", default="topk", choices=["topk", "centroid"],
                    help="topk: the metric's selection; centroid: centroid heads + bank lookup + gate AND up")
    ap.add_argument("--centroids", type=int, default=512, help="centroid vocabulary per head (centroid selection)")
    ap.add_argument("--predictor", default="mlp", choices=["mlp", "trunk"],
                    help="centroid selection: head logits from the two-layer predictor (mlp) or from the paper's own "
                         "predictor, projection blocks -> residual trunk -> heads (trunk; one sequence)")
    return ap.parse_args()


def fnum(v):
    """float for the JSON line; None where a stage was not timed."""
    v = float(v)
    return None if v != v else v


def u16(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            with open(p) as f:
                return float(json.load(f)["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc, self.thread = index, [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0]))
                smax.append(float(r[1]))
            except ValueError:
                continue
            for name, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def oracle_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return 1


def host_mem_available() -> int:
    try:
        with open("/proc/meminfo") as f:
            for line in f:
                if line.startswith("MemAvailable:"):
                    return int(line.split()[1]) * 1024
    except OSError:
        pass
    return 0


def plan_store_layers(cfg, requested: str, world: int):
    """Layers of records the host store holds.  'auto': the whole stack when a host of this size can hold
    and pin it beside everything else (at most half of what is available, per replica), else as many
    layers as that allows; the stack then reads layer l mod Lp (shapes and traffic unchanged)."""
    L = cfg.n_layers
    if requested != "auto":
        n = int(requested)
        return (L if n <= 0 else min(L, n)), "requested"
    layer_bytes = cfg.d_ffn * cfg.record_bytes
    avail = host_mem_available()
    if avail <= 0 or L * layer_bytes <= avail // (2 * max(1, world)):
        return L, "whole store"
    return max(1, min(L, int(avail // (2 * max(1, world)) // layer_bytes))), f"host has {avail / 2**30:.0f} GiB available"


def make_workload(cfg, gen_device: str, pin: bool, store_layers=None):
    """Weights (CPU + generator device), the record store on the host, hidden states."""
    t0 = time.time()
    w1, w2 = synth.predictor_weights(cfg, gen_device)
    if store_layers is not None and store_layers < cfg.n_layers:
        store = torch.empty((store_layers, cfg.d_ffn, 3, cfg.d_model), dtype=torch.bfloat16)
        if pin:
            from paper_2608_22643_b200 import binding as nb
            nb.pin_host_tensor(store)
        synth.fill_backing_store(cfg.with_(n_layers=store_layers), store, gen_device)
        return w1, w2, store, time.time() - t0
    store = torch.empty((cfg.n_layers, cfg.d_ffn, 3, cfg.d_model), dtype=torch.bfloat16)
    if pin:
        from paper_2608_22643_b200 import binding as nb
        nb.pin_host_tensor(store)
    synth.fill_backing_store(cfg, store, gen_device)
    return w1, w2, store, time.time() - t0


def make_pinned_workload(cfg, Lp, lp_why, floor_layers=0, may_shrink=True, make=None):
    """make_workload with a page-locked store of Lp layers.  The host may refuse to page-lock a store that
    MemAvailable said would fit (a limit on locked memory, a fragmented host): then the store is aliased over
    three quarters of the layers, and so on down to an eighth of the stack (or the dense prefix, which must be
    whole).  Returns (w1, w2, store, seconds, layers held, why)."""
    make = make or make_workload
    while True:
        try:
            w1, w2, store, gen_s = make(cfg, "cuda", pin=True, store_layers=Lp)
            return w1, w2, store, gen_s, Lp, lp_why
        except RuntimeError as e:
            if "cudaHostRegister" not in str(e) or not may_shrink or Lp <= max(1, floor_layers, cfg.n_layers // 8):
                raise
            if torch.cuda.is_available():
                torch.cuda.synchronize()
            lp_why = f"the host refused to page-lock {Lp} layers ({Lp * cfg.d_ffn * cfg.record_bytes / 2**30:.0f} GiB)"
            Lp = max(floor_layers, max(1, cfg.n_layers // 8), (3 * Lp) // 4)


def run_oracle_steps(cfg, policy, w1, w2, store, xs, n_steps, layers=None):
    """Times the oracle, as it stands, on steps 1..n_steps of the sequence (step 0 is
    the cold start and is run untimed).  Returns seconds per timed step."""
    from oracle import np_oracle as O
    L = cfg.n_layers if layers is None else layers
    eng = O.Engine(L, cfg.d_model, cfg.d_ffn, cfg.d_pred, cfg.top_k, cfg.capacity,
                   O.EVICT_LRU if policy == "lru" else O.EVICT_EXACT, u16(w1),
                   u16(w2)[: L * cfg.d_ffn], u16(store)[:L])
    eng.step(u16(xs[0]))
    times = []
    for t in range(1, n_steps + 1):
        t0 = time.perf_counter()
        eng.step(u16(xs[t % xs.shape[0]]))
        times.append(time.perf_counter() - t0)
    return times


def reference_arm(args):
    """The oracle timed on the host cores, on this arm's config and metric."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = synth.CONFIGS[args.config]
    if args.rho is not None:
        cfg = cfg.with_(rho=args.rho)
    gen_device = "cuda" if torch.cuda.is_available() else "cpu"
    w1, w2, store, _ = make_workload(cfg, gen_device, pin=False)
    w1, w2 = w1.cpu(), w2.cpu()
    K, W = args.steps, args.warmup
    xs = synth.hidden_states(cfg, K + W + 2)
    # one full step to size the sample: keep the whole run within ~150 s of oracle work
    probe = run_oracle_steps(cfg, args.policy, w1, w2, store, xs, 1)[0]
    budget = 150.0
    L = cfg.n_layers
    layers = L
    if probe * (K + W) > budget:
        layers = max(1, min(L, int(L * budget / (probe * (K + W)))))
    from oracle import np_oracle as O
    eng = O.Engine(layers, cfg.d_model, cfg.d_ffn, cfg.d_pred, cfg.top_k, cfg.capacity,
                   O.EVICT_LRU if args.policy == "lru" else O.EVICT_EXACT, u16(w1),
                   u16(w2)[: layers * cfg.d_ffn], u16(store)[:layers])
    eng.step(u16(xs[0]))                       # cold start, untimed
    for t in range(1, W + 1):
        eng.step(u16(xs[t]))
    t0 = time.perf_counter()
    for t in range(W + 1, W + 1 + K):
        eng.step(u16(xs[t]))
    elapsed = time.perf_counter() - t0
    scale = L / layers                         # a step over `layers` of L layers, scaled to the stack
    ms = elapsed / K * 1000.0 * scale
    value = 1000.0 / ms
    cores = oracle_threads()
    sample = (f"{K} steady-state decode steps of the {cfg.name} stack, first {layers} of {L} layers"
              + (", time scaled by L/layers" if layers != L else ""))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": K, "warmup": W, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: L={L} D={cfg.d_model} M={cfg.d_ffn} H={cfg.d_pred} "
                               f"k={cfg.top_k} C={cfg.capacity} B=1 rho={cfg.rho} policy={args.policy}"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def init_replicas(backend: str, device=None):
    """torch.distributed for N > 1 (None for a single process).  Ranks are independent
    replicas: the only traffic is the barrier and the max-reduction of the timings."""
    if int(os.environ.get("WORLD_SIZE", "1")) <= 1:
        return None
    import torch.distributed as dist
    if device is not None:
        dist.init_process_group(backend, device_id=device)
    else:
        dist.init_process_group(backend)
    return dist


def replica_config(cfg, rank: int):
    """Every replica decodes its own sequence over its own stack."""
    return cfg.with_(seed=cfg.seed + 1000 * rank)


def max_over_ranks(dist, values, device):
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def finish_replicas(dist):
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def cuda_arm(args):
    from paper_2608_22643_b200 import binding as nb
    from paper_2608_22643_b200 import build as nbuild

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (there is no CPU fallback; use --impl reference)")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    dist = init_replicas("nccl", torch.device(dev))
    if rank == 0:
        nbuild.build()
    if dist:
        dist.barrier()
    nb.load()

    cfg = synth.CONFIGS[args.config]
    if args.rho is not None:
        cfg = cfg.with_(rho=args.rho)
    if args.capacity_pct is not None:
        cfg = cfg.with_(capacity_pct=args.capacity_pct)
    cfg = replica_config(cfg, rank)
    K, W = args.steps, args.warmup
    if W < 3:
        raise SystemExit("bench.py: --warmup must be >= 3")
    policy = nb.NP_EVICT_LRU if args.policy == "lru" else nb.NP_EVICT_EXACT
    mode = {"runs": nb.NP_XFER_MEMCPY_RUNS, "gather": nb.NP_XFER_HOST_GATHER,
            "zerocopy": nb.NP_XFER_ZERO_COPY, "file": nb.NP_XFER_FILE}[args.transfer]
    if args.transfer == "file" and args.records != "bf16":
        raise SystemExit("bench.py: --transfer file reads bf16 records")

    if args.budget_gib is not None:
        plan_cfg = nb.make_config(cfg.n_layers, cfg.d_model, cfg.d_ffn, cfg.d_pred, cfg.top_k, cfg.capacity)
        args.dense_layers = nb.np_plan_dense_prefix(plan_cfg, int(args.budget_gib * 2**30), 0)
        if args.dense_layers < 0:
            raise SystemExit("bench.py: the budget does not even hold the sparse layers' resident buffers")
    Lp, lp_why = plan_store_layers(cfg, args.store_layers, int(os.environ.get("LOCAL_WORLD_SIZE", world)))
    if Lp < cfg.n_layers and (args.transfer == "file" or args.dense_layers > Lp):
        raise SystemExit("bench.py: an aliased store is not combined with --transfer file or a longer dense prefix here")
    w1, w2, store, gen_s, Lp, lp_why = make_pinned_workload(cfg, Lp, lp_why, floor_layers=args.dense_layers,
                                                            may_shrink=args.transfer != "file" and args.store_layers == "auto")
    # replicas share one host: the packing threads of the gather transfer are divided among them
    if args.host_threads == 0 and world > 1:
        args.host_threads = nb.replica_host_threads(int(os.environ.get("LOCAL_WORLD_SIZE", world)))
    if args.records == "int8":
        qstore = torch.empty((Lp, cfg.d_ffn, 3 * cfg.d_model + 16), dtype=torch.uint8)
        nb.pin_host_tensor(qstore)
        qstore = synth.quantize_store(store, device="cuda", out=qstore)
        nb.unpin_host_tensor(store)                    # the bf16 store is not used any more
        store = qstore
    ncfg = nb.make_config(cfg.n_layers, cfg.d_model, cfg.d_ffn, cfg.d_pred, cfg.top_k, cfg.capacity,
                          record_format=nb.NP_REC_INT8 if args.records == "int8" else nb.NP_REC_BF16,
                          max_batch=args.batch, evict_policy=policy, transfer_mode=mode,
                          staging_rows=2 * cfg.top_k, chain_layers=args.chain_layers,
                          host_threads=args.host_threads, dense_layers=args.dense_layers, io_depth=args.io_depth,
                          store_layers=Lp if Lp < cfg.n_layers else 0, spec_rows=args.spec_rows,
                          flags=(nb.NP_F_LAYER_LAUNCHES if args.layer_launches or args.direct_loads else 0)
                          | {"auto": 0, "cluster-rows": nb.NP_F_CLUSTER_ROWS, "row-chain": nb.NP_F_ROW_CHAIN}[args.mlp_kernel]
                          | (nb.NP_F_DIRECT_LOADS if args.direct_loads else 0)
                          | (nb.NP_F_TCGEN05_BATCH if args.batch_up_kernel == "tcgen05" else 0)
                          | (nb.NP_F_MAPPED_STAGING if args.mapped_staging else 0))
    storage = None
    if args.transfer == "file":
        # the store goes to a file and leaves host memory; the library sees only the descriptor
        import tempfile
        store_path = args.store_path or os.path.join(tempfile.gettempdir(), f"np_store_{cfg.name}_{os.getpid()}.bin")
        t0 = time.time()
        store.view(torch.int16).numpy().tofile(store_path)
        fd = os.open(store_path, os.O_RDONLY)
        os.fsync(fd)
        os.posix_fadvise(fd, 0, 0, os.POSIX_FADV_DONTNEED)       # reads come from the device, not the page cache
        os.close(fd)
        write_s = time.time() - t0
        store_bytes = store.numel() * 2
        nb.unpin_host_tensor(store)
        store = None
        eng = nb.Engine(ncfg, w1, w2, None, device=dev, store_path=store_path, direct=not args.buffered)
        # the file's own ceiling: one contiguous range of up to 2 GiB through the same reader
        probe_recs = int(min(store_bytes, 2 << 30) // cfg.record_bytes)
        probe = np.empty(probe_recs * cfg.record_bytes + 4096, dtype=np.uint8)
        probe = probe[(-probe.ctypes.data) % 4096:][:probe_recs * cfg.record_bytes]
        t0 = time.time()
        _, used_ring = nb.np_read_records(eng.store_fd, 0, cfg.record_bytes, np.arange(probe_recs), probe, args.io_depth)
        seq_s = time.time() - t0
        del probe
        storage = {"path": store_path, "file_bytes": int(store_bytes), "write_s": write_s, "direct_io": eng.direct_io,
                   "io_uring": bool(used_ring), "io_depth": args.io_depth if args.io_depth else 256,
                   "sequential_read_gbs": probe_recs * cfg.record_bytes / seq_s / 1e9}
    else:
        eng = nb.Engine(ncfg, w1, w2, store, device=dev)
    L, D, M = cfg.n_layers, cfg.d_model, cfg.d_ffn
    rec = cfg.record_bytes                             # resident (bf16) bytes of a record
    rec_store = 3 * D + 16 if args.records == "int8" else rec   # bytes of a record in the store
    reps_timed = max(1, -(-args.min_timed_steps // K))   # the K steps are repeated until the timed region is long enough
    KT = K * reps_timed
    T = 1 + W + KT                                     # cold start + warm-up + timed
    n_detail = 16
    Bq = args.batch
    xs_host = synth.hidden_states(cfg, T + n_detail, batch=Bq, gamma=args.gamma).pin_memory()  # [T + n_detail, B, D] bf16
    xs_dev = xs_host.to(dev)
    out = torch.empty((Bq, D), dtype=torch.float32, device=dev)
    out_host = torch.empty((Bq, D), dtype=torch.float32).pin_memory()
    x_stage = torch.empty((Bq, D), dtype=torch.bfloat16, device=dev)
    s, cs = eng.stream, eng.copy_stream
    centroid = args.selection == "centroid"
    if centroid:
        Kc = args.centroids
        w2c = synth.centroid_head_weights(cfg, Kc, "cuda")
        bank = synth.centroid_bank(cfg, Kc).to(dev)
        head_logits = torch.empty((Bq, L, 2, Kc), dtype=torch.float32, device=dev)
        sel_words = torch.empty((L, M // 32), dtype=torch.int32, device=dev)
    trunk = centroid and args.predictor == "trunk"
    if trunk:
        if Bq != 1:
            raise SystemExit("bench.py: --predictor trunk runs one sequence")
        # The paper's predictor at its sizes (T = 512, four blocks), one gate and one up head per layer
        # of this stack.  Its five layer-0 features are stand-ins made from the step's hidden state
        # (no model is available): the state itself, its LayerNorm, its first 128 values, its RMS, and
        # the arg-max of a fixed random projection as the layer-0 gate centroid ID.
        tT, tK0, tE = 512, 512, 2048
        tdims = (D, D, 128, 1)
        tw = synth.trunk_weights(tT, tdims, tK0, tE, 4, L, Kc, cfg.seed, device="cuda")
        tdesc, ttable = nb.trunk_pack(tw, L)
        tws = torch.empty(nb.np_trunk_workspace_floats(tdesc), dtype=torch.float32, device=dev)
        xf = xs_host[:, 0].to(torch.float32)                                  # [T + n_detail, D]
        gproj = torch.randn(D, tK0, generator=torch.Generator().manual_seed(cfg.seed + 5)) / D ** 0.5
        rms = xf.pow(2).mean(dim=1, keepdim=True).sqrt()
        feats_host = [xf.contiguous(), torch.nn.functional.layer_norm(xf, (D,)).contiguous(), xf[:, :128].contiguous(),
                      torch.cat([rms, torch.zeros(xf.shape[0], 7)], dim=1).contiguous()]
        feats_host = [f.pin_memory() for f in feats_host]
        ids_host = (xf @ gproj).argmax(dim=1).to(torch.int32).pin_memory()
        feats_dev = [f.to(dev) for f in feats_host]
        ids_dev = ids_host.to(dev)
        feat_stage = [torch.empty_like(f[0], device=dev) for f in feats_host]
        id_stage = torch.empty(1, dtype=torch.int32, device=dev)
        trunk_in_bytes = sum(f[0].numel() * 4 for f in feats_host) + 4

    def step(x, feats=None, cid=None):
        if not centroid:
            return nb.np_step(eng.ctx, x, Bq, out, s, cs)
        # the same path with the selection stage swapped: head logits -> arg-max centroids ->
        # bank lookup -> gate AND up -> delta -> install -> MLP chain, all through the C ABI
        if trunk:
            nb.np_trunk_forward(tdesc, ttable, feats, cid, tws, head_logits, s)
        else:
            nb.np_predict_logits_noalloc(eng.w1, w2c, x, Bq, L, D, 2 * Kc, cfg.d_pred, head_logits, s)
        nb.np_centroid_select(eng.ctx, head_logits, Bq, Kc, bank, None, sel_words, s)
        return nb.np_step_selected(eng.ctx, x, Bq, sel_words, out, s, cs)

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    def run_resident(t_lo, t_hi, stats=None):
        for t in range(t_lo, t_hi):
            if trunk:
                step(xs_dev[t], [f[t] for f in feats_dev], ids_dev[t:t + 1])
            else:
                step(xs_dev[t])
            if stats is not None:
                stats.append(eng.counters().copy())

    # ---- device-resident timing ("value") ----------------------------------------------
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    c0.record(s)
    run_resident(0, 1)                                  # cold start: every predicted row of every layer is installed
    c1.record(s)
    run_resident(1, 1 + W)                              # warm-up
    barrier()
    cold_ms = c0.elapsed_time(c1)
    eng.counters()                                      # raises if a kernel reported a fault or a timed-out wait
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = nb.np_launch_count(eng.ctx)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(s)
    run_resident(1 + W, T)
    e1.record(s)
    barrier()
    launches = nb.np_launch_count(eng.ctx) - launches0
    ms_total = e0.elapsed_time(e1)
    eng.counters()

    nd = args.dense_layers
    # ---- per-stage detail on a few more steady-state steps (untimed region) ----------------
    stage_us, delta_rows, overlap, overflow_steps, active_max, spec_rows_seen = [], [], [], 0, 0, []
    for i in range(n_detail):
        t = T + i                                       # the sequence simply continues
        if trunk:
            step(xs_dev[t], [f[t] for f in feats_dev], ids_dev[t:t + 1])
        else:
            step(xs_dev[t])
        stage_us.append(nb.np_last_step_times(eng.ctx))      # centroid selection: the predict stage is outside the call
        c = eng.counters()
        if args.spec_rows and not centroid:
            spec_rows_seen.append(float(np.mean([eng.speculative_lists(l)[0].size for l in range(nd, L)])))
        delta_rows.append(float(c[nd:, nb.NP_CNT_DELTA].mean()) if nd < L else 0.0)
        overflow_steps += int((c[:, nb.NP_CNT_OVERFLOW] > 0).any())
        active_max = max(active_max, int(c[nd:, nb.NP_CNT_ACTIVE].max()) if nd < L else 0)
        overlap.append(float((c[nd:, nb.NP_CNT_KEPT] / np.maximum(1, c[nd:, nb.NP_CNT_PRED])).mean()) if nd < L else 1.0)
    stage_all = np.stack(stage_us)
    step_each = stage_all[:, 0] + stage_all[:, 1] + stage_all[:, 3]   # predict + delta + chain (which waits for the installs)
    stage_us = np.median(stage_all, axis=0)
    n_active = float(eng.counters()[nd:, nb.NP_CNT_ACTIVE].mean()) if nd < L else 0.0

    # ---- end-to-end timing: hidden state from pinned host, result back to the host --------
    nb.np_reset(eng.ctx, s)
    def run_e2e(t_lo, t_hi):
        for t in range(t_lo, t_hi):
            with torch.cuda.stream(s):
                x_stage.copy_(xs_host[t], non_blocking=True)
                if trunk:
                    for dst, src in zip(feat_stage, feats_host):
                        dst.copy_(src[t], non_blocking=True)
                    id_stage.copy_(ids_host[t:t + 1], non_blocking=True)
            if trunk:
                step(x_stage, feat_stage, id_stage)
            else:
                step(x_stage)
            with torch.cuda.stream(s):
                out_host.copy_(out, non_blocking=True)
            s.synchronize()                              # the caller consumes the result every step
    run_e2e(0, 1 + W)
    barrier()
    t0 = time.perf_counter()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g0.record(s)
    run_e2e(1 + W, T)
    g1.record(s)
    barrier()
    e2e_ms_total = g0.elapsed_time(g1)
    clocks = sampler.stop()

    # ---- dominant kernel: the sparse MLP, timed alone on its own stream ---------------------
    reps = 20
    k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        nb.np_mlp_chain(eng.ctx, xs_dev[T - 1], Bq, out, s)
    s.synchronize()
    k0.record(s)
    for _ in range(reps):
        nb.np_mlp_chain(eng.ctx, xs_dev[T - 1], Bq, out, s)
    k1.record(s)
    s.synchronize()
    n_launch = nb.np_chain_launches(eng.ctx)                        # resident launches the chain was cut into
    if n_launch <= 0:
        n_launch = L - nd                                           # per-layer (or batch) kernels
    mlp_kernel = nb.np_mlp_kernel_name(eng.ctx, Bq)       # the kernel the library chose for this shape and batch
    if Bq > 1:
        mlp_kernel += " (the launches of one layer)"
    mlp_us = k0.elapsed_time(k1) * 1000.0 / (reps * n_launch)      # per launch, gaps included
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p0.record(s)
    for _ in range(reps):
        if trunk:
            nb.np_trunk_forward(tdesc, ttable, [f[T - 1] for f in feats_dev], ids_dev[T - 1:T], tws, head_logits, s)
        elif centroid:
            nb.np_predict_logits_noalloc(eng.w1, w2c, xs_dev[T - 1], Bq, L, D, 2 * Kc, cfg.d_pred, head_logits, s)
            nb.np_centroid_select(eng.ctx, head_logits, Bq, Kc, bank, None, sel_words, s)
        else:
            nb.np_predict(eng.ctx, xs_dev[T - 1], Bq, None, None, s)
    p1.record(s)
    s.synchronize()
    pred_us = p0.elapsed_time(p1) * 1000.0 / reps

    # max over ranks
    ms_total, e2e_ms_total = max_over_ranks(dist, [ms_total, e2e_ms_total], dev)

    peak, peak_kind = measured_peaks()
    layer_bytes = n_active * rec + 4 * n_active + 8 * D          # rows + slot list + x in, y out
    mlp_bytes = layer_bytes * L / n_launch                       # one launch spans L / n_launch layers
    if nd:
        # with a dense prefix the figure covers the whole chain: d whole layers + the sparse rest
        n_launch = 1
        mlp_us = k0.elapsed_time(k1) * 1000.0 / reps
        mlp_bytes = nd * (M * rec + 8 * D) + (L - nd) * layer_bytes
        mlp_kernel = "whole MLP chain (dense prefix + sparse layers)"
    achieved = mlp_bytes / (mlp_us * 1e-6) / 1e9
    # DRAM bytes per layer of the dominant kernel from its ncu capture, by kernel and shape; a kernel or
    # shape without a capture reports null rather than another kernel's figure
    per_layer, traffic_src = NCU_TRAFFIC.get((mlp_kernel, cfg.name), (None, None))
    traffic = per_layer * L / n_launch if per_layer is not None and not nd else None
    pred_rows = L * 2 * args.centroids if centroid else L * M
    pred_bytes = 2 * cfg.d_pred * D + 2 * pred_rows * cfg.d_pred + 4 * pred_rows
    if trunk:   # every matrix of the predictor once, plus the logits
        pred_bytes = 2 * (sum(blk[0].numel() for blk in tw["proj"]) + tw["cproj"][0].numel() + tw["heads"].numel()
                          + sum(b[0].numel() + b[4].numel() for b in tw["blocks"])) + 4 * pred_rows
    mean_delta = float(np.mean(delta_rows))
    mean_spec = float(np.mean(spec_rows_seen)) if spec_rows_seen else 0.0
    result = {
        "metric": METRIC, "value": KT * world / (ms_total / 1000.0), "unit": UNIT, "n_gpus": world,
        "steps": K, "warmup": W, "ms_per_step": ms_total / KT, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {
            "workload": f"{cfg.name}: L={L} D={D} M={M} H={cfg.d_pred} k={cfg.top_k} C={cfg.capacity} "
                        f"B={Bq} rho={cfg.rho} policy={args.policy} transfer={args.transfer}"
                        + (f" selection=centroid K={args.centroids}" if centroid else "")
                        + (" predictor=trunk(T=512, 4 blocks)" if trunk else "")
                        + (" records=int8" if args.records == "int8" else "")
                        + (" mapped_staging" if args.mapped_staging else "")
                        + (f" dense_layers={args.dense_layers}" if args.dense_layers else "")
                        + (f" spec_rows={args.spec_rows}" if args.spec_rows else "")
                        + (f" (longest prefix within {args.budget_gib} GiB)" if args.budget_gib is not None else ""),
            "l2": "inputs exceed L2 (per step 866 MB of rows + 365 MB of predictor weights stream through a 126 MB L2)",
            "overlap_measured": float(np.mean(overlap)), "delta_rows_per_layer": mean_delta,
            "speculative_rows_per_layer": mean_spec, "active_rows_per_layer": n_active, "active_rows_max": active_max, "overflow_steps": int(overflow_steps),
            "replicas": world,
            "timed_steps": KT,   # --steps repeated (the sequence continues) so that the timed region is not a few ms
            "store": (f"host store holds all {L} layers" if Lp == L else
                      f"host store aliased over {Lp} of {L} layers (layer l reads layer l mod {Lp}; {lp_why}); shapes, "
                      f"rows and bytes per step are those of the {L}-layer stack"),
            "host_threads": int(args.host_threads),
        },
        "e2e": {"value": KT * world / (e2e_ms_total / 1000.0), "unit": UNIT,
                "h2d_bytes_per_step": int(Bq * D * 2 + (mean_delta + mean_spec) * (L - nd) * rec_store + (trunk_in_bytes if trunk else 0)),
                "d2h_bytes_per_step": int(Bq * D * 4)},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": {"bound": "hbm", "kernel": mlp_kernel, "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_kind": peak_kind + " copy bandwidth (burst)",
                     "traffic": traffic, "traffic_source": traffic_src if traffic is not None else None,
                     "us_per_launch": mlp_us, "bytes_per_launch": mlp_bytes,
                     "layers_per_launch": L / n_launch},
        "stages_us": {"predict_topk": fnum(stage_us[0]), "delta": fnum(stage_us[1]),
                      "install_copy_stream": fnum(stage_us[2]), "mlp_chain_incl_waits": fnum(stage_us[3]),
                      "predict_alone": pred_us, "predict_gbs": pred_bytes / (pred_us * 1e-6) / 1e9,
                      "mlp_chain_alone": mlp_us * n_launch},
        "setup_s": {"generate": gen_s},
        "cold_start": {"ms": cold_ms, "note": "step 0, reported apart from the steady state: empty buffers, every "
                                               "predicted row of every sparse layer crosses to the device"},
    }
    if not centroid:
        # spread over the detail steps, and the step without any transfer (context: what the GPU work alone takes)
        result["step_us"] = {"p10": fnum(np.percentile(step_each, 10)), "median": fnum(np.median(step_each)),
                             "p90": fnum(np.percentile(step_each, 90)), "steps": int(n_detail)}
        compute_us = pred_us + float(stage_us[1]) + mlp_us * n_launch
        result["compute_only"] = {"us": compute_us, "steps_per_s": 1e6 / compute_us,
                                  "note": "predict + delta + MLP chain timed alone, rows already resident: no install"}
    if storage is not None:
        # bytes the step reads from the file over the time the install takes on the copy stream
        storage["read_gbs_during_install"] = mean_delta * (L - nd) * rec / (float(stage_us[2]) * 1e-6) / 1e9
        result["storage"] = storage

    # ---- pinned host -> device copy rate of this machine, measured in the run: the ceiling of the install stage ----
    h2d_gbs = None
    if store is not None:
        probe_bytes = int(min(256 << 20, store.numel() * store.element_size()))
        probe_src = store.view(torch.uint8).view(-1)[:probe_bytes]        # the head of the pinned store, contiguous
        probe_dst = torch.empty(probe_bytes, dtype=torch.uint8, device=dev)
        best = float("inf")
        for _ in range(4):
            h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            h0.record(s)
            with torch.cuda.stream(s):
                probe_dst.copy_(probe_src, non_blocking=True)
            h1.record(s)
            s.synchronize()
            best = min(best, h0.elapsed_time(h1))
        h2d_gbs = probe_bytes / (best * 1e-3) / 1e9
        del probe_dst
        install_bytes = mean_delta * (L - nd) * rec_store
        inst_us = float(stage_us[2])
        if inst_us > 0:
            result["roofline_install"] = {
                "bound": "pcie", "achieved": install_bytes / (inst_us * 1e-6) / 1e9, "peak": h2d_gbs, "unit": "GB/s",
                "frac": install_bytes / (inst_us * 1e-6) / 1e9 / h2d_gbs,
                "peak_kind": f"one contiguous {probe_bytes >> 20} MiB copy from the pinned store, best of 4, in this run",
                "bytes_per_step": install_bytes, "us_per_step": inst_us,
                "note": "the step's bound: scattered records of REC bytes cross to the device while the GPU work "
                        "(compute_only) takes a fraction of the step"}

    # ---- the same step in other settings (reported beside, not as, the value) ----
    if (args.transfer == "gather" and not args.no_variants and not centroid and Bq == 1
            and args.config == "7b" and not (args.layer_launches or args.direct_loads) and not args.dense_layers
            and args.records == "bf16" and world == 1 and args.policy == "exact" and not args.spec_rows):
        eng.close()

        def variant(note, vstore=None, **kw):
            vkw = dict(max_batch=Bq, evict_policy=policy, transfer_mode=mode, staging_rows=2 * cfg.top_k,
                       chain_layers=args.chain_layers, host_threads=args.host_threads,
                       store_layers=Lp if Lp < cfg.n_layers else 0)
            vkw.update(kw)
            vcfg = nb.make_config(cfg.n_layers, cfg.d_model, cfg.d_ffn, cfg.d_pred, cfg.top_k, cfg.capacity, **vkw)
            veng = nb.Engine(vcfg, w1, w2, store if vstore is None else vstore, device=dev)
            vs, vcs = veng.stream, veng.copy_stream
            for t in range(0, 1 + W):
                nb.np_step(veng.ctx, xs_dev[t], Bq, out, vs, vcs)
            barrier()
            z0, z1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            z0.record(vs)
            for t in range(1 + W, T):
                nb.np_step(veng.ctx, xs_dev[t], Bq, out, vs, vcs)
            z1.record(vs)
            barrier()
            cnt = veng.counters()
            veng.close()
            (z_ms,) = max_over_ranks(dist, [z0.elapsed_time(z1)], dev)
            return {"value": KT * world / (z_ms / 1000.0), "unit": UNIT, "ms_per_step": z_ms / KT,
                    "delta_rows_per_layer": float(cnt[:, nb.NP_CNT_DELTA].mean()), "note": note}

        result["variants"] = {
            "transfer=zerocopy": variant("scatter kernel reads the pinned store over PCIe by neuron ID; no host packing, "
                                         "no staging copy", transfer_mode=nb.NP_XFER_ZERO_COPY),
            "policy=lru": variant("rows stay resident while capacity allows (least recently predicted leave first): "
                                  "fewer incoming rows per step than under Eq. 3's exact replacement",
                                  evict_policy=nb.NP_EVICT_LRU),
        }
        qstore = torch.empty((store.shape[0], cfg.d_ffn, 3 * cfg.d_model + 16), dtype=torch.uint8)
        nb.pin_host_tensor(qstore)
        qstore = synth.quantize_store(store, device="cuda", out=qstore)
        result["variants"]["records=int8"] = variant(
            "8-bit row records (int8 rows + fp32 scales), dequantised to bf16 at install: half the bytes cross to the "
            "device; a different workload (the weights are the dequantised ones)", vstore=qstore,
            record_format=nb.NP_REC_INT8)
        nb.unpin_host_tensor(qstore)
        del qstore
        eng = None

    if (rank == 0 and not args.no_cpu_baseline and world == 1 and Bq == 1 and not centroid and not args.dense_layers
            and args.records == "bf16" and store is not None and Lp == cfg.n_layers):
        n = args.cpu_baseline_steps
        times = run_oracle_steps(cfg, args.policy, w1.cpu(), w2.cpu(), store, xs_host, n)
        sec = float(np.mean(times))
        result["cpu_baseline"] = {
            "value": 1.0 / sec, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
            "sample": f"{n} steady-state decode steps of the same stack (all {L} layers), after an untimed cold start"}
    elif rank == 0:
        result["cpu_baseline"] = None
    if eng is not None:
        eng.close()
    if storage is not None and not args.store_path:
        os.remove(storage["path"])
    if rank == 0:
        print(json.dumps(result))
    finish_replicas(dist)


def main():
    args = parse_args()
    if args.impl == "reference":
        reference_arm(args)
    else:
        cuda_arm(args)


if __name__ == "__main__":
    main()
