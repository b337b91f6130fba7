#!/usr/bin/env python
"""Benchmark of the split + Huffman codec on B200.

One *step* = one pass of the whole hot path over the whole synthetic workload: for every tensor
split+histogram on the GPU, codebook on the host, compress on the GPU, decompress on the GPU.
The default workload is the BF16 Llama-8B-shaped weight stack (225 tensors, 15.0 GB).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--chunk-kib C]

Prints ONE JSON line (rank 0).  `value` is uncompressed GB per second through the whole path with all
inputs resident in HBM; `decode` / `encode` / `histogram` hold the per-call throughputs and their
fraction of the HBM roofline time (uncompressed + compressed bytes) / peak; `e2e` repeats the step with
host buffers (pinned) and the host<->device copies inside the timed region; `cpu_baseline` times the CPU
oracle on a bounded sample.  `--impl reference` times the CPU oracle alone (the paper ships no code).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2508_19263_b200 import workloads as wl

METRIC = "decode & encode GB/s (uncompressed bytes) on 1 B200, % HBM roofline, compression ratio"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
ORACLE_SAMPLE_BYTES = int(os.environ.get("ZC_ORACLE_SAMPLE_BYTES", 768 << 20))   # bytes the oracle is timed on (tests shrink it)
# DRAM bytes (read + write) per uncompressed byte from the ncu captures summarised under profiles/ (two-layer BF16
# stack of 872.4 MB, 4 KiB chunks, batched kernels); traffic grows in proportion to the input, so the figure for a
# launch over the whole stack is this ratio times its input bytes.  The write part is undercounted in a capture
# because some of the output is still in L2 when the kernel ends.
NCU_DRAM_BYTES_PER_INPUT_BYTE = {"decode_kernel": (607251968.0 + 827155200.0) / 872415232.0,
                                 "encode_kernel": (872882944.0 + 535107840.0) / 872415232.0}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (no MEASURED_PEAKS.json)"


# --------------------------------------------------------------------------------------------
# workloads
# --------------------------------------------------------------------------------------------

def workload_specs(name: str):
    if name == "cfg2_bf16_llama8b":
        return wl.BF16, wl.llama8b_stack(2)
    if name == "cfg3_fp8_llama8b":
        return wl.FP8_E4M3, wl.llama8b_stack(3)
    if name == "cfg4_fp4_llama8b":
        return wl.FP4_E2M1, wl.llama8b_stack(4)
    if name == "cfg4_fp4_scales":
        # the E8M0 block scales of the same stack as byte streams (config 4 stores them raw; coding them is
        # what the paper's FP4 result rests on, Sec. 3.4 / 4.4): 225 streams, 234.5 MB
        return wl.SCALE_U8, wl.llama8b_stack(4)
    if name in ("cfg5_kv_bf16_all", "cfg5_kv_fp8_all"):
        # config 5 in full: K and V of all 32 layers, [8, 8, 32768, 128] each (34.4 GB in BF16, 17.2 GB in FP8)
        fmt = wl.BF16 if "bf16" in name else wl.FP8_E4M3
        return fmt, [wl.TensorSpec(f"kv.{l}.{'kv'[w]}", (8, 8, 32768, 128), 0.0, 10 * l + w) for l in range(32) for w in range(2)]
    if name in ("cfg5_kv_bf16", "cfg5_kv_fp8", "next3_kv_bf16_static", "next3_kv_fp8_static"):
        # K/V cache tensors [8, 8, 32768, 128]; a subset of the 32 layers keeps the run short (K and V of 4 layers).
        # The *_static workloads code them the way Sec. 3.3 describes the run-time use: with dictionaries computed
        # ahead of time (from layer 0's K and V), no histogram pass and no codebook build in the step
        fmt = wl.BF16 if "bf16" in name else wl.FP8_E4M3
        return fmt, [wl.TensorSpec(f"kv.{l}.{'kv'[w]}", (8, 8, 32768, 128), 0.0, 10 * l + w) for l in range(4) for w in range(2)]
    if name in ("next2_bf16_delta_frozen", "small_bf16_delta_frozen"):
        # the same pair of checkpoints with a stated share of the weights left untouched (frozen layers and rows, the
        # state Sec. 3.1 describes for a fine-tuning run that has converged): unchanged stretches XOR to zero, their
        # chunks are constant and cost no payload bits
        return wl.BF16, wl.llama8b_stack(2) if name.startswith("next2") else wl.llama8b_stack(2, n_layers=2, include_embedding=False)
    if name in ("next2_bf16_delta", "small_bf16_delta"):
        # delta checkpoints (Sec. 3.1 / 4.1): the XOR of two consecutive BF16 checkpoints of the config-2 stack is
        # coded; the earlier checkpoint is a second resident input of every call
        return wl.BF16, wl.llama8b_stack(2) if name.startswith("next2") else wl.llama8b_stack(2, n_layers=2, include_embedding=False)
    if name == "next4_fp8_e5m2":
        # config 3's stack in the other FP8 format (Sec. 3.2 names E5M2, Sec. 4.2 leaves it out): cast without scales
        return wl.FP8_E5M2, wl.llama8b_stack(3)
    if name == "small_bf16":
        return wl.BF16, wl.llama8b_stack(2, n_layers=2, include_embedding=False)
    if name == "small_fp8":
        return wl.FP8_E4M3, wl.llama8b_stack(3, n_layers=2, include_embedding=False)
    raise SystemExit(f"unknown workload {name}")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a timed region runs."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_id: str):
        self.rows = []
        self.proc = None
        self.idx = device_id

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-i", str(self.idx), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        for r in self.rows:
            try:
                sm.append(float(r[1])); mx.append(float(r[2])); power.append(float(r[3]))
                for name, col in (("hw_slowdown", 5), ("hw_thermal_slowdown", 6), ("sw_thermal_slowdown", 7), ("sw_power_cap", 8)):
                    if r[col].lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                continue
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------------------------
# the CPU oracle as baseline / reference arm
# --------------------------------------------------------------------------------------------

def oracle_static_codebook(fmt, sample):
    """The dictionary of the *_static workloads for the oracle legs: from the first tensor of the sample."""
    import oracle as zo
    name, data, n = sample[0]
    return zo.build_codebook(zo.histogram(fmt, data, n), zo.POLICY_STATIC)


def oracle_sample(fmt, specs, device, delta=False):
    """The first tensors of the workload up to ORACLE_SAMPLE_BYTES, as host arrays (delta workloads: the XOR of
    the two checkpoints, which is what the oracle codes)."""
    out, total = [], 0
    for spec in specs:
        if delta:
            cur, base, n = wl.checkpoint_pair(spec, device, frozen_rows=wl.frozen_rows_of(spec) if delta == "frozen" else 0.0)
            t = cur ^ base
        elif spec.name.startswith("kv."):
            t, n = wl.kv_cache_tensor(fmt, spec.seed // 10, spec.seed % 10, device)
        else:
            t, n, _ = wl.make_weight(spec, fmt, device)
        if total and total + t.numel() > ORACLE_SAMPLE_BYTES:
            break
        out.append((spec.name, t.cpu().numpy(), n))
        total += t.numel()
        if total >= ORACLE_SAMPLE_BYTES:
            break
    return out, total


def oracle_step(fmt, sample, chunk_bytes, static_cb=None):
    """Whole path on the CPU oracle (single thread): histogram, codebook, compress, decompress; with a static
    dictionary (Sec. 3.3) the first two fall away."""
    import oracle as zo
    t_h = t_e = t_d = 0.0
    cbytes = 0
    for name, data, n in sample:
        t0 = time.perf_counter()
        if static_cb is None:
            h = zo.histogram(fmt, data, n)
            cb = zo.build_codebook(h, zo.POLICY_AUTO)
        else:
            cb = static_cb
        t1 = time.perf_counter()
        c = zo.compress(fmt, data, n, chunk_bytes, cb)
        t2 = time.perf_counter()
        back = zo.decompress(c, data.size)
        t3 = time.perf_counter()
        assert np.array_equal(back, data)
        t_h += t1 - t0; t_e += t2 - t1; t_d += t3 - t2
        cbytes += c.size
    return t_h, t_e, t_d, cbytes


def cpu_model() -> str:
    try:
        for ln in open("/proc/cpuinfo"):
            if ln.lower().startswith("model name"):
                return ln.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def _oracle_job(job):
    fmt, data, n, chunk_bytes = job
    return oracle_step(fmt, [("slice", data, n)], chunk_bytes)[3]


def oracle_all_cores(fmt, sample, chunk_bytes):
    """The oracle on every core the process may use: the sample is cut into row slices, every slice is compressed
    and decompressed as a tensor of its own by one of N worker processes (N = cores of the affinity mask).
    Returns (GB/s of the whole path, N, slices)."""
    import multiprocessing as mp
    import oracle as zo
    cores = len(os.sched_getaffinity(0))
    per = zo.input_bytes(fmt, zo.group(fmt) * 2) // 2 or 1          # bytes per symbol pair unit: slices stay whole symbols
    jobs = []
    for name, data, n in sample:
        pieces = max(1, min(4 * cores // max(len(sample), 1), data.size // (1 << 20)))
        step = (data.size // pieces) // 64 * 64
        for k in range(pieces):
            lo = k * step
            hi = data.size if k == pieces - 1 else lo + step
            part = data[lo:hi]
            jobs.append((fmt, part, part.size * n // data.size if data.size else 0, chunk_bytes))
    total = sum(j[1].size for j in jobs)
    ctx = mp.get_context("fork")
    t0 = time.perf_counter()
    with ctx.Pool(cores) as pool:
        pool.map(_oracle_job, jobs, chunksize=1)
    return total / (time.perf_counter() - t0) / 1e9, cores, len(jobs)


def run_reference(args):
    """--impl reference: the paper ships no code, so the reference arm is the CPU oracle as it stands."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    fmt, specs = workload_specs(args.workload)
    sample, total = oracle_sample(fmt, specs, "cpu", ("frozen" if args.workload.endswith("_frozen") else True) if "_delta" in args.workload else False)
    chunk_bytes = args.chunk_kib * 1024
    static_cb = oracle_static_codebook(fmt, sample) if args.workload.endswith("_static") else None
    for _ in range(min(args.warmup, 1)):
        oracle_step(fmt, sample[:1], chunk_bytes, static_cb)
    times = []
    for _ in range(args.steps):
        t0 = time.perf_counter()
        t_h, t_e, t_d, cbytes = oracle_step(fmt, sample, chunk_bytes, static_cb)
        times.append(time.perf_counter() - t0)
    dt = float(np.mean(times))
    value = total / dt / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": args.workload, "chunk_kib": args.chunk_kib, "policy": "static" if static_cb else "auto",
                   "sample": f"first {len(sample)} tensors, {total} bytes"},
        "decode": {"value": total / t_d / 1e9, "unit": UNIT}, "encode": {"value": total / t_e / 1e9, "unit": UNIT},
        "compression_ratio": cbytes / total,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": f"first {len(sample)} tensors of {args.workload}, {total} bytes per step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------
# multi-GPU bookkeeping (no data-path collective: every rank compresses its own copy of the workload)
# --------------------------------------------------------------------------------------------

def rank_seed_offset(rank: int) -> int:
    """Weak scaling: every rank holds its own copy of the stack (same shapes, its own seeds)."""
    return 100000 * rank


def max_over_ranks(ms: float, dist, device) -> float:
    """The slowest rank's time; `dist` is torch.distributed (initialised) or None for a single process."""
    if dist is None:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbs(world: int, bytes_per_rank: int, ms: float) -> float:
    """Aggregate throughput of all ranks: every rank processed bytes_per_rank in (at most) ms."""
    return world * bytes_per_rank / ms / 1e6


# --------------------------------------------------------------------------------------------
# the CUDA path
# --------------------------------------------------------------------------------------------

def measure(args, ctx):
    """One workload through the CUDA path: returns the JSON line as a dict (rank 0) or None (other ranks)."""
    from paper_2508_19263_b200 import binding as zc

    rank, world, dev, dist = ctx["rank"], ctx["world"], ctx["dev"], ctx["dist"]

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    fmt, specs = workload_specs(args.workload)
    chunk_bytes = args.chunk_kib * 1024
    # weak scaling: every rank holds its own copy of the stack (same shapes, its own seeds)
    for s in specs:
        s.seed += rank_seed_offset(rank)

    # ---- resident inputs, plans, output buffers ----
    tensors = []
    delta = "_delta" in args.workload
    frozen = args.workload.endswith("_delta_frozen")
    static = args.workload.endswith("_static")
    if static and not args.batch:
        raise SystemExit("the *_static workloads use the batched calls")
    for spec in specs:
        base_t = None
        if delta:
            t, base_t, n = wl.checkpoint_pair(spec, dev, frozen_rows=wl.frozen_rows_of(spec) if frozen else 0.0)
        elif spec.name.startswith("kv."):
            t, n = wl.kv_cache_tensor(fmt, spec.seed // 10, spec.seed % 10, dev)
        else:
            t, n, _ = wl.make_weight(spec, fmt, dev)
        p = zc.plan(fmt, n, chunk_bytes)
        tensors.append({"name": spec.name, "in": t, "base": base_t, "n": n, "plan": p,
                        "comp": torch.empty(p.max_compressed_bytes, dtype=torch.uint8, device=dev),
                        "out": torch.empty(p.input_bytes, dtype=torch.uint8, device=dev),
                        "ws": torch.empty(p.workspace_bytes, dtype=torch.uint8, device=dev)})
    n_t = len(tensors)
    U = sum(t["plan"].input_bytes for t in tensors)
    d_hist = torch.zeros((n_t, 2, 256), dtype=torch.int64, device=dev)
    h_hist = torch.zeros((n_t, 2, 256), dtype=torch.int64).pin_memory()
    stream = torch.cuda.current_stream()
    side = [torch.cuda.Stream(device=dev) for _ in range(max(args.streams - 1, 0))]
    lanes = [stream] + side                      # per-tensor calls go round robin over these streams

    def fork():
        for s in side:
            s.wait_stream(stream)

    def join():
        for s in side:
            stream.wait_stream(s)

    bases = [t["base"] for t in tensors] if delta else None
    hist_batch = zc.HistogramBatch([t["plan"] for t in tensors], [t["in"] for t in tensors], bases)

    def phase_hist():
        if args.batch:
            zc.histogram_batch(hist_batch, d_hist, stream=stream)
            h_hist.copy_(d_hist, non_blocking=True)
            stream.synchronize()
            return
        fork()
        for i, t in enumerate(tensors):
            zc.histogram(t["plan"], t["in"], d_hist[i], stream=lanes[i % len(lanes)], d_base=t["base"])
        join()
        h_hist.copy_(d_hist, non_blocking=True)
        stream.synchronize()

    STATIC_TOLERANCE = 0.05
    dicts = []                                   # *_static: [dictionary of the K tensors, dictionary of the V tensors]

    def phase_codebooks():
        hh = h_hist.numpy()
        if static and dicts:
            for i, t in enumerate(tensors):
                t["cb"] = dicts[i % 2].codebook
            enc_batch.set_codebooks([t["cb"] for t in tensors])
            return
        if args.batch:
            cbs = zc.build_codebooks([t["plan"] for t in tensors], hh, zc.POLICY_AUTO)
            for t, cb in zip(tensors, cbs):
                t["cb"] = cb
            enc_batch.set_codebooks(cbs)
            return
        for i, t in enumerate(tensors):
            t["cb"] = zc.build_codebook(t["plan"], hh[i], zc.POLICY_AUTO)

    enc_batch = zc.CompressBatch([t["plan"] for t in tensors], [t["in"] for t in tensors], [t["comp"] for t in tensors], bases)
    enc_ws = torch.empty(enc_batch.workspace_bytes, dtype=torch.uint8, device=dev)

    def phase_compress():
        if args.batch:
            zc.compress_batch(enc_batch, enc_ws, sync=False, stream=stream)
            return
        fork()
        for i, t in enumerate(tensors):
            zc.compress(t["plan"], t["cb"], t["in"], t["comp"], t["ws"], sync=False, stream=lanes[i % len(lanes)], d_base=t["base"])
        join()

    # every tensor of the stack in one call; the decoder only needs an upper bound of each container's size
    # (the header carries the exact one)
    dec_batch = zc.DecompressBatch([t["plan"] for t in tensors], [t["comp"] for t in tensors],
                                   [t["plan"].max_compressed_bytes for t in tensors], [t["out"] for t in tensors], bases)
    batch_ws = torch.zeros(256, dtype=torch.uint8, device=dev)

    def phase_decompress():
        if args.batch:
            zc.decompress_batch(dec_batch, batch_ws, stream=stream)
            return
        fork()
        for i, t in enumerate(tensors):
            zc.decompress(t["plan"], t["comp"], t["cbytes"], t["out"], t["ws"], stream=lanes[i % len(lanes)], d_base=t["base"])
        join()

    def read_sizes():
        torch.cuda.synchronize()
        for t in tensors:
            hdr = t["comp"][:128].cpu().numpy()
            t["cbytes"] = int(np.frombuffer(hdr[32:40].tobytes(), "<u8")[0])
            t["hdr"] = hdr

    def split_groups(n_groups):
        """Consecutive tensors in n_groups groups of about equal bytes."""
        bounds, acc = [0], 0
        for i, t in enumerate(tensors):
            acc += t["plan"].input_bytes
            if len(bounds) < n_groups and acc >= U * len(bounds) / n_groups:
                bounds.append(i + 1)
        bounds.append(n_t)
        return [list(range(bounds[k], bounds[k + 1])) for k in range(len(bounds) - 1) if bounds[k + 1] > bounds[k]]

    # the step compresses in a few groups: the host builds the codebooks of the next group while the GPU encodes
    step_groups = []
    if args.batch and not static:
        for idx in split_groups(max(1, min(4, n_t // 2))):
            sel = [tensors[i] for i in idx]
            eb = zc.CompressBatch([t["plan"] for t in sel], [t["in"] for t in sel], [t["comp"] for t in sel],
                                  [t["base"] for t in sel] if delta else None)
            hb = zc.HistogramBatch([t["plan"] for t in sel], [t["in"] for t in sel], [t["base"] for t in sel] if delta else None)
            step_groups.append({"idx": idx, "enc": eb, "hist": hb, "ev": torch.cuda.Event(),
                                "ws": torch.empty(eb.workspace_bytes, dtype=torch.uint8, device=dev)})

    def step():
        # histogram of every tensor, then codebook / compress / decompress per tensor: the host builds the
        # next codebook while the GPU is busy with the previous tensors
        if static:
            # run-time use (Sec. 3.3): no histogram, no codebook build; the sizes come back with the call and tell
            # the dictionaries whether they still fit
            sizes = zc.compress_batch(enc_batch, enc_ws, sync=True, stream=stream)
            for i, t in enumerate(tensors):
                if dicts[i % 2].observe(t["plan"].input_bytes, sizes[i]):
                    raise SystemExit(f"dictionary {i % 2} no longer fits tensor {t['name']}")
            zc.decompress_batch(dec_batch, batch_ws, stream=stream)
            return
        if args.batch:
            # group by group: the counts of a group come back while the GPU counts the next one, and the host builds
            # a group's codebooks while the GPU is still busy with histograms or with the group before
            hh = h_hist.numpy()
            for g in step_groups:
                lo, hi = g["idx"][0], g["idx"][-1] + 1
                zc.histogram_batch(g["hist"], d_hist[lo:hi], stream=stream)
                h_hist[lo:hi].copy_(d_hist[lo:hi], non_blocking=True)
                g["ev"].record(stream)
            for g in step_groups:
                lo, hi = g["idx"][0], g["idx"][-1] + 1
                g["ev"].synchronize()
                cbs = zc.build_codebooks([tensors[i]["plan"] for i in g["idx"]], hh[lo:hi], zc.POLICY_AUTO)
                for i, cb in zip(g["idx"], cbs):
                    tensors[i]["cb"] = cb
                g["enc"].set_codebooks(cbs)
                zc.compress_batch(g["enc"], g["ws"], sync=False, stream=stream)
            zc.decompress_batch(dec_batch, batch_ws, stream=stream)
            return
        phase_hist()
        hh = h_hist.numpy()
        fork()
        for i, t in enumerate(tensors):
            ln = lanes[i % len(lanes)]
            t["cb"] = zc.build_codebook(t["plan"], hh[i], zc.POLICY_AUTO)
            zc.compress(t["plan"], t["cb"], t["in"], t["comp"], t["ws"], sync=False, stream=ln, d_base=t["base"])
            zc.decompress(t["plan"], t["comp"], t["plan"].max_compressed_bytes, t["out"], t["ws"], stream=ln, d_base=t["base"])
        join()

    def timed(fn, reps):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            fn()
        e1.record(stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), dist, dev) / reps

    C_own = None
    if static:
        # for comparison: the container sizes with every tensor's own codebook
        phase_hist()
        phase_codebooks()
        phase_compress()
        read_sizes()
        C_own = sum(t["cbytes"] for t in tensors)
        hh = h_hist.numpy()
        dicts.extend(zc.Dictionary(tensors[w]["plan"], hh[w], STATIC_TOLERANCE) for w in range(2))
        phase_codebooks()

    # ---- correctness of what is timed (untimed): statuses, byte-identical round trip ----
    step()
    read_sizes()
    for t in tensors:
        st = zc.OK if args.batch else zc.device_status(t["plan"], t["ws"])
        if st != zc.OK:
            raise SystemExit(f"device status {st} on {t['name']}")
        if not torch.equal(t["out"], t["in"]):
            raise SystemExit(f"round trip mismatch on {t['name']}")
    if args.batch:
        bad = [zc.batch_status(w) for w in [batch_ws] + [g["ws"] for g in step_groups] if zc.batch_status(w) != (zc.OK, None)]
        if bad:
            raise SystemExit(f"batch status: {bad}")
    C = sum(t["cbytes"] for t in tensors)

    for _ in range(max(args.warmup - 1, 0)):
        step()

    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        gpu_id = str(local_rank)
    sampler = ClockSampler(gpu_id)
    if rank == 0:
        sampler.start()
    ms_step = timed(step, args.steps)
    # per-call throughputs: the same calls, each kind timed back to back over all tensors
    ms_hist = timed(phase_hist, args.steps)
    phase_codebooks()
    t0 = time.perf_counter()
    phase_codebooks()
    ms_codebook = (time.perf_counter() - t0) * 1e3
    ms_enc = timed(phase_compress, args.steps)
    ms_dec = timed(phase_decompress, args.steps)
    clocks = sampler.stop() if rank == 0 else None

    # ---- end to end with host buffers: H2D of the inputs and D2H of the containers inside the timed region ----
    e2e = None
    try:
        if args.no_e2e:
            raise RuntimeError("skipped (--no-e2e)")
        h_in = [t["in"].cpu().pin_memory() for t in tensors]
        h_out = [torch.empty(t["cbytes"], dtype=torch.uint8).pin_memory() for t in tensors]

        # Batched calls, pipelined over groups of tensors: the H2D copies of all groups are queued on one stream,
        # the kernels of a group start when its inputs have arrived, its containers leave on a third stream, so
        # that both PCIe directions and the GPU work at the same time.
        groups = split_groups(max(1, min(8, n_t // 4)))
        s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        gb = []
        if args.batch:
            for idx in groups:
                sel = [tensors[i] for i in idx]
                gbase = [t["base"] for t in sel] if delta else None
                enc_g = zc.CompressBatch([t["plan"] for t in sel], [t["in"] for t in sel], [t["comp"] for t in sel], gbase)
                gb.append({"idx": idx,
                           "hist": zc.HistogramBatch([t["plan"] for t in sel], [t["in"] for t in sel], gbase),
                           "enc": enc_g, "enc_ws": torch.empty(enc_g.workspace_bytes, dtype=torch.uint8, device=dev),
                           "dec": zc.DecompressBatch([t["plan"] for t in sel], [t["comp"] for t in sel],
                                                     [t["plan"].max_compressed_bytes for t in sel], [t["out"] for t in sel], gbase),
                           "dec_ws": torch.zeros(256, dtype=torch.uint8, device=dev),
                           "ev_in": torch.cuda.Event(), "ev_enc": torch.cuda.Event()})

        def e2e_step():
            if args.batch:
                s_in.wait_stream(stream)
                s_out.wait_stream(stream)
                with torch.cuda.stream(s_in):
                    for g in gb:
                        for i in g["idx"]:
                            tensors[i]["in"].copy_(h_in[i], non_blocking=True)
                        g["ev_in"].record(s_in)
                for g in gb:
                    lo, hi = g["idx"][0], g["idx"][-1] + 1
                    stream.wait_event(g["ev_in"])
                    if static:
                        g["enc"].set_codebooks([tensors[i]["cb"] for i in g["idx"]])
                    else:
                        zc.histogram_batch(g["hist"], d_hist[lo:hi], stream=stream)
                        h_hist[lo:hi].copy_(d_hist[lo:hi], non_blocking=True)
                        stream.synchronize()                   # the host needs the counts for the codebooks
                        cbs = zc.build_codebooks([tensors[i]["plan"] for i in g["idx"]], h_hist[lo:hi].numpy(), zc.POLICY_AUTO)
                        g["enc"].set_codebooks(cbs)
                    zc.compress_batch(g["enc"], g["enc_ws"], sync=False, stream=stream)
                    g["ev_enc"].record(stream)
                    with torch.cuda.stream(s_out):
                        s_out.wait_event(g["ev_enc"])
                        for i in g["idx"]:
                            h_out[i].copy_(tensors[i]["comp"][: tensors[i]["cbytes"]], non_blocking=True)
                    zc.decompress_batch(g["dec"], g["dec_ws"], stream=stream)
                stream.wait_stream(s_in)
                stream.wait_stream(s_out)
                return
            for i, t in enumerate(tensors):
                t["in"].copy_(h_in[i], non_blocking=True)
                zc.histogram(t["plan"], t["in"], d_hist[i], d_base=t["base"])
            h_hist.copy_(d_hist, non_blocking=True)
            stream.synchronize()
            hh = h_hist.numpy()
            for i, t in enumerate(tensors):
                cb = zc.build_codebook(t["plan"], hh[i], zc.POLICY_AUTO)
                zc.compress(t["plan"], cb, t["in"], t["comp"], t["ws"], sync=False, d_base=t["base"])
                h_out[i].copy_(t["comp"][: t["cbytes"]], non_blocking=True)
                zc.decompress(t["plan"], t["comp"], t["plan"].max_compressed_bytes, t["out"], t["ws"], d_base=t["base"])

        e2e_step()
        ms_e2e = timed(e2e_step, max(1, min(args.steps, 3)))
        e2e = {"value": whole_job_gbs(world, U, ms_e2e), "unit": UNIT, "h2d_bytes_per_step": U, "d2h_bytes_per_step": C + n_t * 4096,
               "ms_per_step": ms_e2e,
               "groups": len(gb) if args.batch else n_t,
               "note": ("host tensor -> H2D -> compress with the static dictionaries -> D2H container" if static else
                        "host tensor -> H2D -> histogram -> codebook -> compress -> D2H container")
                       + "; decoded tensor stays on the device; pipelined over groups of tensors on three streams"}
        del h_in, h_out
    except Exception as ex:  # pinned host memory for the whole stack may be unavailable
        e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0, "error": str(ex)[:200]}

    if rank != 0:
        return None

    peak, peak_src = measured_peaks()
    gbs = lambda nbytes, ms: nbytes / ms / 1e6

    def leg(ms, nbytes_alg):
        return {"value": whole_job_gbs(world, U, ms), "unit": UNIT, "ms": ms, "algorithmic_bytes": nbytes_alg,
                "hbm_gbs": gbs(nbytes_alg, ms), "frac_of_measured_peak": gbs(nbytes_alg, ms) / peak,
                "frac_of_nominal_8TBs": gbs(nbytes_alg, ms) / NOMINAL_HBM_GBS}

    # kernel launches of one call of each kind over the whole stack
    if args.batch:
        combos = {}
        for t in tensors:
            key = tuple(t["cb"].modes) if t["n"] else (0, 0)
            combos[key] = combos.get(key, 0) + 1
        n_enc_launch = sum((c + 255) // 256 for c in combos.values())
        n_dec_launch = (n_t + 447) // 448
        n_hist_launch = (n_t + 767) // 768
        # the step encodes group by group: one launch per group and combination of stream modes in it
        n_enc_launch_step = 0
        for g in step_groups:
            gc = {}
            for i in g["idx"]:
                key = tuple(tensors[i]["cb"].modes) if tensors[i]["n"] else (0, 0)
                gc[key] = gc.get(key, 0) + 1
            n_enc_launch_step += sum((c + 255) // 256 for c in gc.values())
    else:
        n_enc_launch = n_dec_launch = n_hist_launch = n_enc_launch_step = n_t
    # delta form: the earlier checkpoint is read once more by every kernel
    B_extra = U if delta else 0
    dec, enc, hist = leg(ms_dec, U + C + B_extra), leg(ms_enc, U + C + B_extra), leg(ms_hist, U + B_extra)
    dom_name, dom = ("decode_kernel", dec) if ms_dec >= ms_enc else ("encode_kernel", enc)
    roofline = {"bound": "hbm", "kernel": dom_name, "achieved": dom["hbm_gbs"], "peak": peak, "unit": "GB/s",
                "frac": dom["hbm_gbs"] / peak, "peak_source": peak_src,
                "launches_per_call": n_dec_launch if dom_name == "decode_kernel" else n_enc_launch,
                "avg_launch_ms": (ms_dec / n_dec_launch if dom_name == "decode_kernel" else ms_enc / n_enc_launch),
                "algorithmic_bytes_per_launch": (U + C) / (n_dec_launch if dom_name == "decode_kernel" else n_enc_launch),
                "traffic": (NCU_DRAM_BYTES_PER_INPUT_BYTE[dom_name] * U / (n_dec_launch if dom_name == "decode_kernel" else n_enc_launch)
                            if args.workload == "cfg2_bf16_llama8b" and args.chunk_kib == 4 and args.batch else None),
                "traffic_source": "from profiles/ (ncu dram__bytes_read+write of the two-layer BF16 stack, scaled by input bytes per launch), not measured in this run"}

    # ---- CPU oracle on a bounded sample of the same workload (rank 0, N=1 only) ----
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        sample, total = oracle_sample(fmt, specs, dev, ('frozen' if frozen else True) if delta else False)
        t_h, t_e, t_d, cb_sample = oracle_step(fmt, sample, chunk_bytes, oracle_static_codebook(fmt, sample) if static else None)
        cpu = {"value": total / (t_h + t_e + t_d) / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"first {len(sample)} tensors of {args.workload}, {total} bytes",
               "decode_gbs": total / t_d / 1e9, "encode_gbs": total / t_e / 1e9, "histogram_codebook_gbs": (total / t_h / 1e9 if not static else None),
               "cpu_model": cpu_model()}
        if not static and not delta:
            try:
                all_gbs, n_cores, n_slices = oracle_all_cores(fmt, sample, chunk_bytes)
                cpu["all_cores"] = {"value": all_gbs, "unit": UNIT, "cores": n_cores,
                                    "sample": f"the same sample cut into {n_slices} row slices, each compressed and decompressed as a tensor of its own by one of {n_cores} worker processes"}
            except Exception as ex:
                cpu["all_cores"] = {"value": None, "error": str(ex)[:200]}

    # compression ratios next to the paper's (context): exponent stream, sign+mantissa stream, total
    st_bits = [0, 0]
    for t in tensors:
        for s in range(2):
            st_bits[s] += int(np.frombuffer(t["hdr"][64 + 32 * s + 16: 64 + 32 * s + 24].tobytes(), "<u8")[0])
    n_syms = sum(t["plan"].n_syms for t in tensors)
    line = {
        "metric": METRIC, "value": whole_job_gbs(world, U, ms_step), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": args.workload, "tensors": n_t, "uncompressed_bytes": U, "compressed_bytes": C,
                   "chunk_kib": args.chunk_kib,
                   "policy": f"static dictionaries from layer 0's K and V, tolerance {STATIC_TOLERANCE}" if static else "auto",
                   "batched_calls": bool(args.batch), "streams": args.streams if not args.batch else 1,
                   "l2": "inputs larger than L2 (no flush)"},
        "decode": dec, "encode": enc, "histogram": hist, "codebook_host_ms": ms_codebook,
        "compression_ratio": {"total_container": C / U, "total_container_own_codebooks": (C_own / U if C_own else None), "exponent_stream_payload": st_bits[0] / (8 * n_syms),
                              "sign_mantissa_stream_payload": st_bits[1] / (8 * n_syms),
                              "paper_context": "abstract: up to 62% (BF16) / 83% (FP8) total"},
        "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "clocks": clocks,
        "gpu_launches": ((n_enc_launch if static else (len(step_groups) if args.batch else n_hist_launch) + n_enc_launch_step)
                         + n_dec_launch) * args.steps,
    }
    return line


# Workloads reported next to the headline (key, workload, chunk KiB): the other configurations the paper's
# method is measured on, the larger chunk sizes, and the rows that follow the headline path.
PER_WORKLOAD = [
    ("cfg3_fp8_llama8b", "cfg3_fp8_llama8b", 4),
    ("cfg5_kv_bf16_32layers", "cfg5_kv_bf16_all", 4),
    ("cfg5_kv_fp8_32layers", "cfg5_kv_fp8_all", 4),
    ("cfg4_fp4_llama8b", "cfg4_fp4_llama8b", 4),
    ("cfg4_fp4_scales", "cfg4_fp4_scales", 4),
    ("cfg2_bf16_llama8b_chunk16k", "cfg2_bf16_llama8b", 16),
    ("cfg2_bf16_llama8b_chunk64k", "cfg2_bf16_llama8b", 64),
    ("cfg3_fp8_llama8b_chunk16k", "cfg3_fp8_llama8b", 16),
    ("cfg3_fp8_llama8b_chunk64k", "cfg3_fp8_llama8b", 64),
    ("next2_bf16_delta", "next2_bf16_delta", 4),
    ("next2_bf16_delta_frozen", "next2_bf16_delta_frozen", 4),
    ("next3_kv_bf16_static", "next3_kv_bf16_static", 4),
    ("next4_fp8_e5m2", "next4_fp8_e5m2", 4),
]


def summary_of(line):
    """What per_workload keeps of a workload's line."""
    out = {"workload": line["config"]["workload"], "chunk_kib": line["config"]["chunk_kib"], "tensors": line["config"]["tensors"],
           "uncompressed_bytes": line["config"]["uncompressed_bytes"], "compressed_bytes": line["config"]["compressed_bytes"],
           "container_ratio": line["compression_ratio"]["total_container"],
           "exponent_stream_ratio": line["compression_ratio"]["exponent_stream_payload"],
           "sign_mantissa_stream_ratio": line["compression_ratio"]["sign_mantissa_stream_payload"],
           "step_ms": line["ms_per_step"], "step_gbs": line["value"], "round_trip": "byte-identical"}
    for leg in ("decode", "encode", "histogram"):
        out[leg] = {k: line[leg][k] for k in ("ms", "value", "hbm_gbs", "frac_of_measured_peak", "frac_of_nominal_8TBs")}
    if line.get("extra"):
        out.update(line["extra"])
    return out


def config1_latency(ctx):
    """Config 1 (one 1024 x 1024 FP8 E4M3 tensor, 64 KiB chunks): a latency case, microseconds per call."""
    from paper_2508_19263_b200 import binding as zc
    dev = ctx["dev"]
    d_in, n = wl.config1_tensor(dev)
    p = zc.plan(wl.FP8_E4M3, n, 65536)
    d_hist = torch.zeros((2, 256), dtype=torch.int64, device=dev)
    d_out = torch.empty(p.max_compressed_bytes, dtype=torch.uint8, device=dev)
    d_back = torch.empty(p.input_bytes, dtype=torch.uint8, device=dev)
    d_ws = torch.empty(p.workspace_bytes, dtype=torch.uint8, device=dev)
    hist = zc.histogram(p, d_in, d_hist).cpu().numpy().astype(np.uint64)
    cb = zc.build_codebook(p, hist, zc.POLICY_HUFF_ALL)          # the config codes both streams
    nbytes = zc.compress(p, cb, d_in, d_out, d_ws)
    zc.decompress(p, d_out, nbytes, d_back, d_ws)
    if zc.device_status(p, d_ws) != zc.OK or not torch.equal(d_back, d_in[: p.input_bytes]):
        raise SystemExit("config 1 round trip mismatch")

    def timed_us(fn, reps=200):
        for _ in range(10):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / reps

    return {"workload": "cfg1_fp8_1024x1024", "chunk_kib": 64, "policy": "huff_all", "uncompressed_bytes": p.input_bytes,
            "compressed_bytes": nbytes, "container_ratio": nbytes / p.input_bytes, "round_trip": "byte-identical",
            "histogram_us": timed_us(lambda: zc.histogram(p, d_in, d_hist)),
            "encode_us": timed_us(lambda: zc.compress(p, cb, d_in, d_out, d_ws, sync=False)),
            "decode_us": timed_us(lambda: zc.decompress(p, d_out, nbytes, d_back, d_ws)),
            "note": "asynchronous calls back to back on one stream, CUDA events; 16 chunks: a latency case, not a bandwidth case"}


def run_ours(args):
    import copy
    import gc
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=dev)
        dist = dist_mod
    ctx = {"rank": rank, "world": world, "dev": dev, "dist": dist}
    line = measure(args, ctx)
    # the other workloads, device-resident legs only, one after the other (single GPU, default workload only)
    if world == 1 and args.per_workload and args.workload == "cfg2_bf16_llama8b" and args.chunk_kib == 4 and args.batch:
        per = {}
        for key, name, ck in PER_WORKLOAD:
            gc.collect(); torch.cuda.empty_cache()
            sub = copy.copy(args)
            sub.workload, sub.chunk_kib, sub.steps, sub.warmup = name, ck, 3, 2
            sub.no_e2e, sub.no_cpu_baseline = True, True
            try:
                per[key] = summary_of(measure(sub, ctx))
            except SystemExit as ex:
                per[key] = {"workload": name, "chunk_kib": ck, "error": str(ex)[:200]}
        gc.collect(); torch.cuda.empty_cache()
        per["cfg1_fp8_1024x1024_chunk64k"] = config1_latency(ctx)
        line["per_workload"] = per
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2_bf16_llama8b")
    ap.add_argument("--chunk-kib", type=int, default=4)
    ap.add_argument("--streams", type=int, default=4,
                    help="CUDA streams the per-tensor calls are spread over (tails of one tensor's kernels overlap the next)")
    ap.add_argument("--batch", type=int, default=1, choices=[0, 1],
                    help="1: the batched entry points (all tensors of the stack per call); 0: one call per tensor")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (used for profiler captures)")
    ap.add_argument("--per-workload", type=int, default=1, choices=[0, 1],
                    help="1: after the headline workload, time the other configurations and add them as per_workload")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
