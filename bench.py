#!/usr/bin/env python
"""Benchmark of the SGNS minibatch step (positive word-context pairs per second).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload large|sponsored|medium|small|tiny]
    python bench.py --impl reference ...      # the CPU checker timed on the host cores

One step = the whole hot path (sub-sampling, compaction, windows, negatives, gather, dots,
coefficients, scatter-add) over one chunk of a seeded synthetic Zipfian token stream, in
Hogwild mode.  Prints ONE JSON line.  With N > 1 (under torchrun) every rank trains its own
replica on its own chunks: there is no data-path collective, only the timing reduction.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1606_08495_b200 import corpus  # noqa: E402

METRIC = "sgns_positive_pairs_per_sec"
UNIT = "pairs/s"
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes moved per algorithmic byte by the update kernels of a Hogwild step on the large workload (the
# launch that draws the step's negatives plus the gather / update kernel), from one one-pass ncu capture of
# those kernels ((dram__bytes_read.sum + dram__bytes_write.sum) / model bytes of the captured step:
# (5.01 + 120.61) / 121.9 GB, rows on 128-byte boundaries).  It is a constant taken once, not a counter read
# during this run (the JSON line says so in "traffic_kind"), and applies to the large workload in Hogwild
# mode with the default row stride and launch shape only; anything else reports null.
TRAFFIC_PER_ALGORITHMIC_BYTE = 1.031


def algorithmic_bytes(d, centres, pairs, negatives):
    """Rows touched by a Hogwild step, 4d bytes each, read once and written once:
    the centre rows plus one output row per target (no credit for cache hits)."""
    return 4 * d * (2 * centres + 2 * pairs * (1 + negatives))


def algorithmic_bytes_snapshot(d, centres, pairs, negatives):
    """Three-pass snapshot plan: pass 1 reads C + T rows, writes C scratch rows and T coefficients;
    pass 2 reads C rows and T coefficients and read-modify-writes T rows; pass 3 reads C scratch rows
    and read-modify-writes C rows (T = pairs * (1 + negatives))."""
    T = pairs * (1 + negatives)
    return 4 * d * (3 * T + 6 * centres) + 8 * T


def algorithmic_bytes_cbow(d, examples, pairs, negatives, snapshot=False):
    """CBOW step: `pairs` context rows (one per (centre, context) pair) and E (1 + N) target rows.
    Hogwild: every row read once and written once.  Snapshot: pass 1 reads P + T rows and writes E
    scratch rows, pass 2 re-reads P rows and read-modify-writes T, pass 3 reads E and
    read-modify-writes P (T = E (1 + N))."""
    T = examples * (1 + negatives)
    if snapshot:
        return 4 * d * (4 * pairs + 3 * T + 2 * examples) + 8 * T
    return 4 * d * (2 * pairs + 2 * T)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def physical_gpu_index(local_rank):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        parts = [p for p in vis.split(",") if p]
        if local_rank < len(parts) and parts[local_rank].isdigit():
            return int(parts[local_rank])
    return local_rank


def row_stride_for(d, requested=0):
    """Floats between table rows: the requested value, else rows padded to 128-byte boundaries."""
    return requested if requested else (d + 31) // 32 * 32


def pick_workload(name, free_bytes, requested_stride=0):
    """The named configuration, else the largest one whose tables fit the GPU."""
    order = ["large", "sponsored", "medium", "small", "tiny"]
    if name:
        return name
    for cand in order:
        c = corpus.CONFIGS[cand]
        need = 2 * c["vocab"] * row_stride_for(c["d"], requested_stride) * 4 + 12 * c["vocab"] + 3 * (1 << 30)
        if need < free_bytes:
            return cand
    return "tiny"


# --------------------------------------------------------------------------------------------
# the CPU checker timed on the host (cpu_baseline leg and --impl reference)
# --------------------------------------------------------------------------------------------
def time_oracle(cfg, cp, sample_words, steps, warmup, first_chunk=500_000):
    from oracle import Oracle

    dense_bytes = 2 * cfg["vocab"] * cfg["d"] * 4
    sparse = dense_bytes > 8 * (1 << 30)
    o = Oracle(cfg["vocab"], cfg["d"], 1, sparse=sparse)
    o.build_tables(cp.counts, cfg["subsample_t"])
    W, N, lr = cfg["window"], cfg["negatives"], cfg["lr"]
    for i in range(warmup):
        o.step(cp.chunk(first_chunk + i, sample_words), W, N, lr, 1)
    pairs, secs = 0, 0.0
    for i in range(steps):
        toks = cp.chunk(first_chunk + warmup + i, sample_words)
        t0 = time.perf_counter()
        st = o.step(toks, W, N, lr, 1)
        secs += time.perf_counter() - t0
        pairs += st["pairs"]
    o.close()
    store = "sparse lazily initialised row store" if sparse else "dense tables"
    return pairs, secs, store


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    name = args.workload or "large"
    cfg = corpus.CONFIGS[name]
    cp = corpus.Corpus(cfg)
    words = args.ref_words
    pairs, secs, store = time_oracle(cfg, cp, words, args.steps, args.warmup)
    value = pairs / secs if secs > 0 else 0.0
    sample = f"{args.steps} steps of a {words}-word prefix of a chunk of the {name} workload, sequential mode, {store}"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": name, "vocab": cfg["vocab"], "d": cfg["d"], "window": cfg["window"],
                   "negatives": cfg["negatives"], "tokens_per_step": words},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------
# the CUDA library
# --------------------------------------------------------------------------------------------
def reduce_over_ranks(ms, e2e_ms, pairs, e2e_pairs, launches, world, device):
    """Whole-job figures from one rank's: the slowest rank's times, work and launches summed."""
    if world <= 1:
        return ms, e2e_ms, pairs, e2e_pairs, launches
    import torch
    import torch.distributed as dist

    vals = torch.tensor([ms, e2e_ms, pairs, e2e_pairs, float(launches)], dtype=torch.float64, device=device)
    mx = vals.clone(); dist.all_reduce(mx, op=dist.ReduceOp.MAX)
    sm = vals.clone(); dist.all_reduce(sm, op=dist.ReduceOp.SUM)
    return float(mx[0]), float(mx[1]), float(sm[2]), float(sm[3]), int(sm[4])


def measured_tensor_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops_sustained"]), "measured sustained bf16"
    except Exception:
        return 1400.0, "fallback sustained bf16"


def fill_clustered(table, rows, d, lo, hi, seed, cluster_size=50, noise=0.55, loose=0.2):
    """Writes the recipe of corpus.clustered_rows into rows [lo, hi) of a device table (torch's
    generator on the device instead of numpy's: same distribution, other numbers).  Input data."""
    import torch

    dev = table.device
    g = torch.Generator(device=dev); g.manual_seed(seed)
    view = table.view(rows, -1)
    n_clusters = max(1, (hi - lo) // cluster_size)
    centres = torch.randn(n_clusters, d, generator=g, device=dev)
    for a in range(lo, hi, 1 << 20):
        b = min(hi, a + (1 << 20))
        which = torch.randint(0, n_clusters, (b - a,), generator=g, device=dev)
        is_loose = torch.rand(b - a, generator=g, device=dev) < loose
        x = noise * torch.randn(b - a, d, generator=g, device=dev)
        x += torch.where(is_loose[:, None], torch.zeros((), device=dev), centres[which])
        x[is_loose] *= 1.0 / noise
        view[a:b, :d] = x


def secondary_modes(model, cfg, dev_chunks, first_step, dev, steps=10, warmup=3):
    """The other modes on the model the headline run leaves in memory: snapshot-mode SGNS steps, CBOW
    Hogwild steps, and one retrieval call over the model's last 3 M rows (overwritten with clustered
    stand-in vectors first, so this runs last).  Each entry: CUDA-event ms per step, the update (or
    retrieval) kernels' time from the library's own events, algorithmic bytes or flops over that time,
    and the fraction of the measured peak."""
    import torch

    from paper_1606_08495_b200 import binding

    W, N, lr, d = cfg["window"], cfg["negatives"], cfg["lr"], cfg["d"]
    peak, peak_kind = measured_peak()
    out = {}
    n_chunks = min(len(dev_chunks), warmup + steps)

    def timed(step_fn, sample_fn, bytes_fn, label):
        counts = []
        for i in range(warmup, n_chunks):
            model.set_step(first_step + i)
            st = binding.StepStats()
            sample_fn(dev_chunks[i], st)
            counts.append((st.centres, st.pairs))
        model.set_step(first_step)
        for i in range(warmup):
            step_fn(dev_chunks[i])
        model.sync()
        binding.w2v_profile_enable(model.h, True)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize(dev)
        ev0.record()
        for i in range(warmup, n_chunks):
            step_fn(dev_chunks[i])
        ev1.record()
        torch.cuda.synchronize(dev)
        ms = ev0.elapsed_time(ev1)
        kernel_ms, _ = binding.w2v_profile_read(model.h)
        binding.w2v_profile_enable(model.h, False)
        k = n_chunks - warmup
        pairs = float(sum(p for _, p in counts))
        nbytes = float(sum(bytes_fn(c, p) for c, p in counts))
        achieved = nbytes / (kernel_ms * 1e-3) / 1e9 if kernel_ms > 0 else 0.0
        out[label] = {"value": pairs / (ms * 1e-3), "unit": UNIT, "steps": k, "ms_per_step": ms / k,
                      "kernel_ms_per_step": kernel_ms / k, "bound": "hbm", "achieved": achieved, "peak": peak,
                      "roofline_unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}"}

    timed(lambda t: binding.w2v_sgns_step(model.h, t, t.numel(), W, N, lr, binding.MODE_SNAPSHOT, None),
          lambda t, st: binding.w2v_sample_pairs(model.h, t, t.numel(), W, N, None, None, None, 0, st,
                                                 allow=(binding.W2V_ERR_CAPACITY,)),
          lambda c, p: algorithmic_bytes_snapshot(d, c, p, N), "sgns_snapshot")
    timed(lambda t: binding.w2v_cbow_step(model.h, t, t.numel(), W, N, lr, binding.MODE_HOGWILD, None),
          lambda t, st: binding.w2v_sample_cbow(model.h, t, t.numel(), W, N, None, None, 0, st,
                                                allow=(binding.W2V_ERR_CAPACITY,)),
          lambda c, p: algorithmic_bytes_cbow(d, c, p, N), "cbow_hogwild")
    out["cbow_hogwild"]["note"] = "pairs = (centre, context) pairs, i.e. context rows read"
    timed(lambda t: binding.w2v_cbow_step(model.h, t, t.numel(), W, N, lr, binding.MODE_SNAPSHOT, None),
          lambda t, st: binding.w2v_sample_cbow(model.h, t, t.numel(), W, N, None, None, 0, st,
                                                allow=(binding.W2V_ERR_CAPACITY,)),
          lambda c, p: algorithmic_bytes_cbow(d, c, p, N, True), "cbow_snapshot")

    free_b, _ = torch.cuda.mem_get_info(dev)
    if free_b > (5 << 30):
        V = cfg["vocab"]
        lo, hi, m, K = V - 3_000_000, V, 8192, 30
        fill_clustered(model.U, V, d, lo, hi, seed=5)
        g = torch.Generator(device=dev); g.manual_seed(6)
        q = torch.randint(lo, hi, (m,), generator=g, device=dev, dtype=torch.int64)
        ids = torch.empty(m * K, dtype=torch.int64, device=dev)
        cs = torch.empty(m * K, dtype=torch.float32, device=dev)
        tpeak, tkind = measured_tensor_peak()
        for tau, label in ((0.65, "topk_cosine_tau_0.65"), (-2.0, "topk_cosine_top30")):
            for _ in range(2):
                binding.w2v_topk_cosine(model.h, 0, q, m, lo, hi, K, tau, ids, cs)
            model.sync()
            binding.w2v_profile_enable(model.h, True)
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize(dev)
            ev0.record()
            calls = 5
            for _ in range(calls):
                binding.w2v_topk_cosine(model.h, 0, q, m, lo, hi, K, tau, ids, cs)
            ev1.record()
            torch.cuda.synchronize(dev)
            model.sync()
            ms = ev0.elapsed_time(ev1)
            kernel_ms, _ = binding.w2v_profile_read(model.h)
            binding.w2v_profile_enable(model.h, False)
            cosines = float(m) * (hi - lo) * calls
            achieved = 2.0 * d * cosines / (kernel_ms * 1e-3) / 1e12 if kernel_ms > 0 else 0.0
            out[label] = {"value": cosines / (ms * 1e-3), "unit": "cosines/s", "steps": calls, "ms_per_step": ms / calls,
                          "kernel_ms_per_step": kernel_ms / calls, "bound": "tensor", "achieved": achieved,
                          "peak": tpeak, "roofline_unit": "TFLOP/s", "frac": achieved / tpeak,
                          "peak_kind": f"of {tkind}",
                          "config": {"queries": m, "candidates": hi - lo, "K": K, "tau": tau,
                                     "rows": "clustered stand-in vectors (cluster centre + noise), lists fill",
                                     "lists_full": float(((ids.view(m, K) >= 0).sum(dim=1) == K).float().mean())}}
    return out


def run_gpu(args):
    import torch
    import torch.distributed as dist

    from paper_1606_08495_b200 import binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    free_b, _ = torch.cuda.mem_get_info(dev)
    name = pick_workload(args.workload, free_b, args.row_stride)
    cfg = corpus.CONFIGS[name]
    if args.tokens_per_step:
        cfg = corpus.scaled(cfg, minibatch=args.tokens_per_step)
    cp = corpus.Corpus(cfg)
    W, N, lr, d = cfg["window"], cfg["negatives"], cfg["lr"], cfg["d"]
    K, Wu = args.steps, args.warmup
    mode = binding.MODE_HOGWILD if args.mode == "hogwild" else binding.MODE_SNAPSHOT
    cbow = args.model == "cbow"
    step_dev = binding.w2v_cbow_step if cbow else binding.w2v_sgns_step
    step_host = binding.w2v_cbow_step_host if cbow else binding.w2v_sgns_step_host

    row_stride = d if args.dense_rows else row_stride_for(d, args.row_stride)
    model = binding.W2V(cfg["vocab"], d, seed=1, device=dev, row_stride=row_stride)
    model.build_alias(cp.counts, cfg["subsample_t"])
    model.set_tuning(args.rows_in_flight, args.blocks_per_sm)

    # every rank reads its own part of the stream: chunk index = rank * stride + i
    stride = 10_000
    n_chunks = Wu + 2 * K
    host_chunks = [torch.from_numpy(cp.chunk(rank * stride + i)).pin_memory() for i in range(n_chunks)]
    dev_chunks = [c.to(dev) for c in host_chunks[: Wu + K]]
    torch.cuda.synchronize(dev)

    # exact counts of the timed steps (same seed and step number as the steps themselves)
    centres, pairs = [], []
    for i in range(Wu, Wu + K):
        model.set_step(i)
        t = dev_chunks[i]
        st = binding.StepStats()
        if cbow:
            binding.w2v_sample_cbow(model.h, t, t.numel(), W, N, None, None, 0, st,
                                    allow=(binding.W2V_ERR_CAPACITY,))
        else:
            binding.w2v_sample_pairs(model.h, t, t.numel(), W, N, None, None, None, 0, st,
                                     allow=(binding.W2V_ERR_CAPACITY,))
        centres.append(st.centres); pairs.append(st.pairs)
    model.set_step(0)

    def barrier():
        if world > 1:
            dist.barrier()

    # ---- device-timed run: inputs already resident in HBM ----
    for i in range(Wu):
        step_dev(model.h, dev_chunks[i], dev_chunks[i].numel(), W, N, lr, mode, None)
    model.sync()
    binding.w2v_profile_enable(model.h, True)
    launches0 = model.launch_count()
    sampler = ClockSampler(physical_gpu_index(local_rank))
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(); torch.cuda.synchronize(dev)
    sampler.start()
    ev0.record()
    IL = max(1, args.interleave)
    for i in range(Wu, Wu + K):
        for phase in range(IL):                       # IL > 1: interleaved minibatches, one step number
            if IL > 1:
                binding.w2v_set_step(model.h, i)
                binding.w2v_set_interleave(model.h, phase, IL)
            step_dev(model.h, dev_chunks[i], dev_chunks[i].numel(), W, N, lr, mode, None)
    ev1.record()
    torch.cuda.synchronize(dev); barrier()
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1)
    launches = model.launch_count() - launches0
    kernel_ms, kernel_launches = binding.w2v_profile_read(model.h)
    binding.w2v_profile_enable(model.h, False)

    # ---- end-to-end run: host chunks in pinned memory, counters read back every step ----
    e2e_pairs = 0
    h2d = d2h = 0
    st = binding.StepStats()
    barrier(); torch.cuda.synchronize(dev)
    ev2, ev3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev2.record()
    for i in range(Wu + K, Wu + 2 * K):
        t = host_chunks[i]
        for phase in range(IL):
            if IL > 1:
                binding.w2v_set_step(model.h, i)
                binding.w2v_set_interleave(model.h, phase, IL)
            step_host(model.h, t, t.numel(), W, N, lr, mode, st)
            e2e_pairs += st.pairs
            h2d += 4 * t.numel(); d2h += 64
    ev3.record()
    torch.cuda.synchronize(dev); barrier()
    e2e_ms = ev2.elapsed_time(ev3)

    tot_pairs = float(sum(pairs))
    if cbow:
        tot_bytes = float(sum(algorithmic_bytes_cbow(d, c, p, N, args.mode == "snapshot") for c, p in zip(centres, pairs)))
    else:
        model_bytes = algorithmic_bytes if args.mode == "hogwild" else algorithmic_bytes_snapshot
        tot_bytes = float(sum(model_bytes(d, c, p, N) for c, p in zip(centres, pairs)))
    ms, e2e_ms, all_pairs, all_e2e_pairs, all_launches = reduce_over_ranks(
        ms, e2e_ms, tot_pairs, float(e2e_pairs), launches, world, dev)

    default_shape = (name == "large" and args.mode == "hogwild" and not cbow and not args.row_stride
                     and not args.rows_in_flight and not args.blocks_per_sm and not args.dense_rows
                     and not args.tokens_per_step and IL == 1)
    # the memory system's own ceiling for the update's access pattern on this table (random rows gathered and
    # added to, no sampling, no arithmetic: w2v_probe_rows), measured right after the timed steps
    ceiling = None
    if rank == 0 and not cbow and args.mode == "hogwild" and d <= 512:
        best, done = None, 0
        for _ in range(3):
            pms, done = binding.w2v_probe_rows(model.h, binding.PROBE_GATHER_RED, cfg["vocab"], min(20_000_000, 40 * cfg["vocab"]))
            best = pms if best is None or pms < best else best
        ceiling = 2.0 * 4 * d * done / (best * 1e-3) / 1e9
    secondary = None
    if world == 1 and default_shape and not args.no_secondary:
        secondary = secondary_modes(model, cfg, dev_chunks, Wu + 2 * K, dev)

    if rank == 0:
        peak, peak_kind = measured_peak()
        achieved = tot_bytes / (kernel_ms * 1e-3) / 1e9 if kernel_ms > 0 else 0.0
        groups = K          # one group of update kernels per step (1 launch in hogwild mode, 3-4 in snapshot mode)
        per_launch_bytes = tot_bytes / max(1, groups)
        line = {
            "metric": METRIC, "value": all_pairs / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": Wu, "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": name, "vocab": cfg["vocab"], "d": d, "window": W, "negatives": N,
                       "subsample_t": cfg["subsample_t"], "tokens_per_step": int(dev_chunks[0].numel()),
                       "model": args.model, "mode": args.mode, "row_stride_floats": row_stride, "interleave": IL, "parallelism": f"replicas x{world}" if world > 1 else "1 gpu",
                       "l2": "tables and gathers far larger than L2 (random rows of %.1f GB)" % (2 * cfg["vocab"] * d * 4 / 1e9)
                             if 2 * cfg["vocab"] * d * 4 > 4 * 126e6 else "tables fit in L2; no flush between steps",
                       "pairs_per_step": tot_pairs / K, "centres_per_step": sum(centres) / K,
                       "trained_pairs_incl_negatives_per_sec": all_pairs * (1 + N) / (ms * 1e-3),
                       "centres_per_sec": world * sum(centres) / (ms * 1e-3)},
            "clocks": clocks,
            "e2e": {"value": all_e2e_pairs / (e2e_ms * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": h2d // K, "d2h_bytes_per_step": d2h // K},
            "gpu_launches": all_launches,
            "roofline": {"bound": "hbm",
                         "kernel": ("cbow_hogwild_kernel" if cbow and args.mode == "hogwild" else "cbow_snap_* (3 passes)" if cbow
                                    else "draw_negatives_kernel + sgns_hogwild_kernel" if args.mode == "hogwild"
                                    else "draw_negatives_kernel + sgns_snap_* (3 passes)"),
                         "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                         "frac_of_8TBps": achieved / 8000.0,
                         "algorithmic_bytes_per_launch": per_launch_bytes,
                         "kernel_ms_per_launch": kernel_ms / max(1, groups),
                         "access_pattern_ceiling": (None if ceiling is None else
                                                    {"what": "random rows of the same table gathered and added to (w2v_probe_rows), GB/s of row bytes",
                                                     "GBps": ceiling, "achieved_over_ceiling": achieved / ceiling}),
                         "traffic": (TRAFFIC_PER_ALGORITHMIC_BYTE * per_launch_bytes if default_shape else None),
                         "traffic_kind": ("scaled from one ncu capture of this kernel and workload, not measured in this run"
                                          if default_shape else None)},
        }
        if secondary is not None:
            line["secondary"] = secondary
        if world == 1 and not args.no_cpu_baseline:
            words = args.cpu_words
            p, s, store = time_oracle(cfg, cp, words, 1, 0)
            line["cpu_baseline"] = {
                "value": p / s if s > 0 else 0.0, "unit": UNIT, "cores": 1, "kind": "oracle",
                "sample": f"one step over a {words}-word prefix of a chunk of the {name} workload "
                          f"({p} pairs, {s:.1f} s), sequential mode, {store}"}
        print(json.dumps(line), flush=True)
    model.close()
    if world > 1:
        dist.destroy_process_group()


def algorithmic_bytes_sharded(d, centres, pairs, negatives, shards):
    """Column-sharded step, summed over the shards (their slice widths add up to d): dotprod reads
    C + T slice rows; adjust reads T rows for the centre sums, writes and re-reads C scratch rows,
    reads C rows and read-modify-writes T rows, then read-modify-writes C rows.  Each shard also adds
    its T partial dots into `shards` arrays (8 B each) and moves 16 B per target of dots and
    coefficients."""
    T = pairs * (1 + negatives)
    return 4 * d * (4 * T + 6 * centres) + (8 * shards * shards + 16 * shards) * T


def run_sharded(args):
    """The paper's column partition: `--shards S` shards of one model, here all on one GPU, one after
    another (the step a rank of an S-GPU run executes is one shard's share of this)."""
    import torch

    from paper_1606_08495_b200 import binding
    from paper_1606_08495_b200.sharded import LocalShards

    if int(os.environ.get("WORLD_SIZE", "1")) != 1:
        raise SystemExit("--mode sharded times the shards of one model on one GPU; run it without torchrun")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    S = args.shards
    free_b, _ = torch.cuda.mem_get_info(dev)
    name = args.workload
    if not name:
        for cand in ["large", "sponsored", "medium", "small", "tiny"]:
            c = corpus.CONFIGS[cand]
            if 2 * c["vocab"] * c["d"] * 4 + 12 * S * c["vocab"] + 8 * (1 << 30) < free_b:
                name = cand
                break
    cfg = corpus.CONFIGS[name]
    cp = corpus.Corpus(cfg)
    W, N, lr, d = cfg["window"], cfg["negatives"], cfg["lr"], cfg["d"]
    K, Wu = args.steps, args.warmup
    from paper_1606_08495_b200.sharded import shard_columns
    widest = max(hi - lo for lo, hi in shard_columns(d, S))
    aligned = (not args.dense_rows and
               2 * cfg["vocab"] * binding.aligned_row_stride(widest) * 4 * S + 12 * S * cfg["vocab"] + 8 * (1 << 30) < free_b)
    model = LocalShards(cfg["vocab"], d, 1, S, device=dev, aligned_rows=aligned, exchange=args.exchange)
    model.build_alias(cp.counts, cfg["subsample_t"])
    chunks = [torch.from_numpy(cp.chunk(i)).to(dev) for i in range(Wu + K)]
    for i in range(Wu):
        model.step(chunks[i], W, N, lr)
    model.sync()
    for m in model.models:
        binding.w2v_profile_enable(m.h, True)
    launches0 = model.launch_count()
    sampler = ClockSampler(physical_gpu_index(0))
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(dev)
    sampler.start()
    ev0.record()
    centres, pairs = [], []
    for i in range(Wu, Wu + K):
        st = model.step(chunks[i], W, N, lr)
        centres.append(st["centres"]); pairs.append(st["pairs"])
    ev1.record()
    torch.cuda.synchronize(dev)
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1)
    launches = model.launch_count() - launches0
    per_shard_ms = [binding.w2v_profile_read(m.h)[0] for m in model.models]
    kernel_ms = sum(per_shard_ms)
    tot_pairs = float(sum(pairs))
    tot_bytes = float(sum(algorithmic_bytes_sharded(d, c, p, N, S) for c, p in zip(centres, pairs)))
    peak, peak_kind = measured_peak()
    achieved = tot_bytes / (kernel_ms * 1e-3) / 1e9 if kernel_ms > 0 else 0.0
    line = {
        "metric": METRIC, "value": tot_pairs / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": K, "warmup": Wu,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": name, "vocab": cfg["vocab"], "d": d, "window": W, "negatives": N,
                   "mode": "sharded", "shards": S, "columns": model.columns,
                   "rows": "on 128-byte boundaries" if aligned else "dense", "exchange": args.exchange,
                   "parallelism": f"{S} column shards run one after another on 1 gpu",
                   "pairs_per_step": tot_pairs / K,
                   "slowest_shard_ms_per_step": max(per_shard_ms) / K,
                   "exchange_bytes_per_shard_and_step": 4.0 * tot_pairs / K * (1 + N),
                   "pairs_per_sec_if_each_shard_had_its_own_gpu_exchange_excluded": tot_pairs / (max(per_shard_ms) * 1e-3)},
        "clocks": clocks, "gpu_launches": launches,
        "roofline": {"bound": "hbm", "kernel": "shard_dots + coefficients + shard_du + snapshot passes 2-3",
                     "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": f"of {peak_kind}", "algorithmic_bytes_per_launch": tot_bytes / K,
                     "kernel_ms_per_launch": kernel_ms / K, "traffic": None},
    }
    print(json.dumps(line), flush=True)
    model.close()


def run_topk(args):
    """Retrieval by cosine similarity (Section 2 / Section 7.2): K = 30 nearest above tau = 0.65 for a
    batch of query rows among the last 15 % of the vocabulary (the share of the ad ids in the
    sponsored-search-shaped workload).  One step = one w2v_topk_cosine call."""
    import torch

    from paper_1606_08495_b200 import binding

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    name = args.workload or "sponsored"
    cfg = corpus.CONFIGS[name]
    V, d = cfg["vocab"], cfg["d"]
    K, tau, m = 30, args.tau, args.queries
    lo, hi = int(V * 0.85), V
    model = binding.W2V(V, d, seed=1, device=dev, row_stride=row_stride_for(d, args.row_stride))
    tensor = args.retrieval_kernel != "fp32"
    binding.w2v_set_retrieval_kernel(model.h, {"fp32": 0, "tensor": 1, "screen": 2, "pairs": 3}[args.retrieval_kernel])
    # stand-in for trained vectors: clustered rows (centre + noise), so that queries have neighbours above
    # tau and the lists fill; --unrelated-rows keeps the earlier i.i.d. normal rows (nothing reaches tau = 0.65:
    # pure screening).  Written by torch: this is input data.
    g = torch.Generator(device=dev); g.manual_seed(5)
    if args.unrelated_rows:
        Uv = model.U.view(V, model.row_stride)
        for a in range(0, V, 1 << 20):
            b = min(V, a + (1 << 20))
            Uv[a:b, :d] = torch.randn(b - a, d, generator=g, device=dev)
    else:
        fill_clustered(model.U, V, d, 0, V, seed=5)
    q = torch.randint(0, V, (m,), generator=g, device=dev, dtype=torch.int64)
    ids = torch.empty(m * K, dtype=torch.int64, device=dev)
    cs = torch.empty(m * K, dtype=torch.float32, device=dev)
    Ksteps, Wu = args.steps, args.warmup
    for _ in range(Wu):
        binding.w2v_topk_cosine(model.h, 0, q, m, lo, hi, K, tau, ids, cs)
    model.sync()
    binding.w2v_profile_enable(model.h, True)
    launches0 = model.launch_count()
    sampler = ClockSampler(physical_gpu_index(0))
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(dev)
    sampler.start()
    ev0.record()
    for _ in range(Ksteps):
        binding.w2v_topk_cosine(model.h, 0, q, m, lo, hi, K, tau, ids, cs)
    ev1.record()
    torch.cuda.synchronize(dev)
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1)
    kernel_ms, _ = binding.w2v_profile_read(model.h)
    launches = model.launch_count() - launches0
    # end to end: query ids from pinned host memory, results back to the host
    qh = q.cpu().pin_memory()
    ids_h = torch.empty(m * K, dtype=torch.int64).pin_memory()
    cs_h = torch.empty(m * K, dtype=torch.float32).pin_memory()
    ev2, ev3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev2.record()
    for _ in range(Ksteps):
        q.copy_(qh, non_blocking=True)
        binding.w2v_topk_cosine(model.h, 0, q, m, lo, hi, K, tau, ids, cs)
        ids_h.copy_(ids, non_blocking=True); cs_h.copy_(cs, non_blocking=True)
    ev3.record()
    torch.cuda.synchronize(dev)
    e2e_ms = ev2.elapsed_time(ev3)
    cosines = float(m) * (hi - lo) * Ksteps
    flops = 2.0 * d * cosines
    sm_mhz = clocks.get("sm_max_mhz") or 1965.0
    achieved = flops / (kernel_ms * 1e-3) / 1e12 if kernel_ms > 0 else 0.0
    if tensor:
        # useful flops against the tensor peak of the type the MMAs run in: measured dense bf16 x the
        # nominal tf32 / bf16 ratio (1.1 / 2.25 PFLOP/s); each useful product costs three TF32 MMAs
        try:
            with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
                bf16, kind = float(json.load(f)["bf16_tflops_sustained"]), "measured sustained bf16 x 1.1/2.25"
        except Exception:
            bf16, kind = 1400.0, "fallback sustained bf16 x 1.1/2.25"
        bound = "tensor"
        mma_per_product = 3 if args.retrieval_kernel == "tensor" else 1
        if mma_per_product == 3:
            peak = bf16 * 1.1 / 2.25
            peak_kind = kind + " (tf32); the kernel issues 3 MMA flops per useful flop"
        else:
            peak = bf16        # the screen's MMAs are bf16 x bf16 -> fp32
            peak_kind = kind.replace(" x 1.1/2.25", "") + "; one bf16 MMA flop per useful flop, plus fp32 dot products for the candidates near the cut"
    else:
        peak, bound = 148 * 128 * 2 * sm_mhz * 1e6 / 1e12, "alu"     # fp32 FMA lanes x 2 flop x clock, TFLOP/s
        peak_kind = "148 SMs x 128 fp32 FMA lanes x 2 flop x max SM clock"
    line = {
        "metric": "cosine_similarities_per_sec", "value": cosines / (ms * 1e-3), "unit": "cosines/s", "n_gpus": 1,
        "steps": Ksteps, "warmup": Wu, "ms_per_step": ms / Ksteps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": name + " (retrieval)", "vocab": V, "d": d, "queries_per_step": m,
                   "candidates": hi - lo, "K": K, "tau": tau, "row_stride_floats": model.row_stride,
                   "kernel": {"tensor": "tcgen05 tf32, head/tail split (3 MMAs per product)",
                              "screen": "tcgen05 bf16 screen (1 MMA per product) + exact fp32 cosines near the cut",
                              "pairs": "the same screen with cta_group::2 MMAs on pairs of SMs",
                              "fp32": "fp32 CUDA cores"}[args.retrieval_kernel],
                   "rows": "i.i.d. normal (no neighbours)" if args.unrelated_rows else "clustered (centre + noise): lists fill",
                   "lists_full": float(((ids.view(m, K) >= 0).sum(dim=1) == K).float().mean()),
                   "l2": "3 M candidate rows (3.8 GB) streamed per call, far larger than L2"},
        "clocks": clocks,
        "e2e": {"value": cosines / (e2e_ms * 1e-3), "unit": "cosines/s", "h2d_bytes_per_step": 8 * m,
                "d2h_bytes_per_step": 12 * m * K},
        "gpu_launches": launches,
        "roofline": {"bound": bound, "kernel": {"tensor": "topk_cosine_tc_kernel", "screen": "topk_cosine_screen_kernel",
                                                "pairs": "topk_cosine_screen_pair_kernel",
                                                "fp32": "topk_cosine_kernel"}[args.retrieval_kernel],
                     "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                     "mma_tflops_issued": mma_per_product * achieved if tensor else None,
                     "peak_kind": peak_kind,
                     "flops_per_launch": flops / Ksteps, "kernel_ms_per_launch": kernel_ms / Ksteps, "traffic": None},
    }
    print(json.dumps(line), flush=True)
    model.close()


def run_probe(args):
    """Memory-system ceilings for the step's access patterns (w2v_probe_rows) on the output table of
    the chosen workload's model: each pattern with row numbers spread over the whole table and over
    the first `--probe-span` rows only (the table is the same; only the address range differs)."""
    import torch

    from paper_1606_08495_b200 import binding

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    free_b, _ = torch.cuda.mem_get_info(dev)
    name = pick_workload(args.workload, free_b, args.row_stride)
    cfg = corpus.CONFIGS[name]
    cp = corpus.Corpus(cfg)
    d = cfg["d"]
    row_stride = d if args.dense_rows else row_stride_for(d, args.row_stride)
    model = binding.W2V(cfg["vocab"], d, seed=1, device=dev, row_stride=row_stride)
    model.build_alias(cp.counts, cfg["subsample_t"])
    peak, peak_kind = measured_peak()
    names = ["gather", "gather_red", "gather_alias", "gather_red_alias", "touch_red"]
    rows = args.probe_rows
    spans = sorted({cfg["vocab"], min(cfg["vocab"], args.probe_span)}, reverse=True)
    result = {}
    for span in spans:
        per = {}
        for access, label in enumerate(names):
            best = None
            for _ in range(1 + max(1, args.steps // 10)):          # first launch is the warm-up
                ms, done = binding.w2v_probe_rows(model.h, access, span, rows)
                best = ms if best is None or ms < best else best
            moved = done * 4.0 * d * (2.0 if "red" in label else 1.0)
            per[label] = {"ms": best, "row_GBps": moved / (best * 1e-3) / 1e9, "frac_of_copy_peak": moved / (best * 1e-3) / 1e9 / peak}
        result[f"span_{span}_rows"] = per
    # the ring of bulk copies that feeds the retrieval kernels: GB/s per SM against stage size, depth and producer lanes
    ring = {}
    for stage, stages, producers in ((16384, 8, 1), (16384, 4, 1), (32768, 4, 1), (49152, 3, 1), (16384, 8, 2), (8192, 16, 1)):
        best = None
        for _ in range(3):
            ms, done = binding.w2v_probe_bulk_ring(model.h, stage, stages, producers, 64 << 20)
            best = ms if best is None or ms < best else best
        model.sync()
        ring[f"{stage}B_x{stages}_stages_{producers}_producer"] = {"ms": best, "GBps_per_sm": done / (best * 1e-3) / 1e9,
                                                                   "ns_per_stage": best * 1e6 / (done / stage)}
    # producer lanes, ring and MMA issuer coupled, without an epilogue: SM cycles per 19-MMA tile (2432 at the pipe's rate)
    feed = {}
    tiles = int(min(3900, cfg["vocab"] * row_stride * 4 // 3 // 163840))
    for kps, stages, span in ((3, 3, 0), (3, 3, 1), (2, 4, 0), (2, 4, 1), (4, 2, 1), (1, 9, 0)):
        cyc, waited = binding.w2v_probe_mma_ring(model.h, kps, stages, tiles, span)
        feed[f"{kps}_kblocks_x{stages}_stages_{'spanning_tiles' if span else 'per_tile'}"] = {"cycles_per_tile": cyc, "of_them_waiting_for_data": waited}
    line = {"metric": "random_row_traffic", "unit": "GB/s of row bytes (read + written)", "n_gpus": 1,
            "bulk_copy_ring": ring, "mma_ring_cycles_per_tile": feed,
            "config": {"workload": name + " (memory-system probe)", "vocab": cfg["vocab"], "d": d,
                       "row_stride_floats": row_stride, "rows_per_launch": rows,
                       "table_GB": cfg["vocab"] * row_stride * 4 / 1e9},
            "peak": peak, "peak_kind": f"of {peak_kind}", "probe": result}
    print(json.dumps(line), flush=True)
    model.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", choices=list(corpus.CONFIGS), default=None)
    ap.add_argument("--rows-in-flight", type=int, default=0)
    ap.add_argument("--blocks-per-sm", type=int, default=0)
    ap.add_argument("--row-stride", type=int, default=0,
                    help="floats between table rows (0 = d rounded up to a multiple of 32, i.e. rows on 128-byte "
                         "boundaries; pass d itself for dense rows)")
    ap.add_argument("--cpu-words", type=int, default=150_000, help="word tokens in the cpu_baseline sample")
    ap.add_argument("--ref-words", type=int, default=20_000, help="word tokens per step of --impl reference")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--queries", type=int, default=8192, help="query rows per call of --mode topk")
    ap.add_argument("--retrieval-kernel", choices=["fp32", "tensor", "screen", "pairs"], default="screen")
    ap.add_argument("--tau", type=float, default=0.65, help="similarity threshold of --mode topk (-2 keeps everything)")
    ap.add_argument("--probe-rows", type=int, default=20_000_000, help="--mode probe: rows touched per launch")
    ap.add_argument("--probe-span", type=int, default=18_000_000,
                    help="--mode probe: the second measurement draws its rows from the first this-many rows only")
    ap.add_argument("--mode", choices=["hogwild", "snapshot", "sharded", "topk", "probe"], default="hogwild",
                    help="update mode of the timed steps (the headline number is hogwild); sharded = the "
                         "paper's column partition, --shards slices of one model on one GPU")
    ap.add_argument("--tokens-per-step", type=int, default=0,
                    help="word tokens per chunk (0 = the workload's own minibatch)")
    ap.add_argument("--shards", type=int, default=8)
    ap.add_argument("--model", choices=["sgns", "cbow"], default="sgns",
                    help="skip-gram (the headline) or the continuous-bag-of-words variant; for cbow the "
                         "metric counts (centre, context) pairs, i.e. context rows read")
    ap.add_argument("--interleave", type=int, default=1,
                    help="visit every chunk this many times, each time with 1/this of its input words "
                         "(interleaved minibatch formation)")
    ap.add_argument("--dense-rows", action="store_true", help="no padding between table rows")
    ap.add_argument("--no-secondary", action="store_true",
                    help="default run only: skip the snapshot / CBOW / retrieval measurements that follow the headline")
    ap.add_argument("--unrelated-rows", action="store_true",
                    help="--mode topk: i.i.d. normal rows (no neighbours above tau) instead of clustered ones")
    ap.add_argument("--exchange", choices=["p2p", "allreduce"], default="p2p",
                    help="--mode sharded: partial dots added into every shard's array by the producing kernel, "
                         "or stored per shard and summed afterwards")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        print("note: fewer than 3 warm-up steps; not a valid timing", file=sys.stderr)
    if args.impl == "reference":
        run_reference(args)
    elif args.mode == "sharded":
        run_sharded(args)
    elif args.mode == "topk":
        run_topk(args)
    elif args.mode == "probe":
        run_probe(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
