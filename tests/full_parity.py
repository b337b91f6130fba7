"""Bit-exact parity of the CUDA path with the CPU oracle over EVERY tensor of a bench workload at full size.

The pytest suite compares complete containers on small tensors and sampled chunks at bench size; this script is
the exhaustive pass: for each tensor of the workload the GPU's histogram, container bytes and decoded bytes are
compared with the oracle's histogram, its container (its own codebook from its own histogram) and the input.
The oracle side runs in worker processes (one tensor each), the GPU side in the calling process through the
batched C-ABI calls.

    python tests/full_parity.py --workload cfg2_bf16_llama8b --chunk-kib 4 --procs 16

Prints one line per workload and exits non-zero on the first difference.
"""
import argparse
import os
import shutil
import sys
import tempfile
import time
from concurrent.futures import ProcessPoolExecutor, wait, FIRST_COMPLETED
import multiprocessing as mp

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def oracle_check(fmt, n_elems, chunk_bytes, data_path, cont_path, hist_gpu):
    """Worker process: the oracle's whole path on one tensor against what the GPU produced."""
    import oracle as zo
    data = np.load(data_path, mmap_mode="r")
    cont = np.load(cont_path, mmap_mode="r")
    data = np.ascontiguousarray(data)
    hist = zo.histogram(fmt, data, n_elems)
    if not np.array_equal(hist, hist_gpu):
        return "histogram differs"
    want = zo.compress(fmt, data, n_elems, chunk_bytes, zo.build_codebook(hist, zo.POLICY_AUTO))
    if want.size != cont.size or not np.array_equal(want, cont):
        return f"container differs (oracle {want.size} bytes, GPU {cont.size} bytes)"
    if not np.array_equal(zo.decompress(np.ascontiguousarray(cont), data.size), data):
        return "the oracle does not decode the GPU's container to the input"
    os.unlink(data_path)
    os.unlink(cont_path)
    return None


def run(workload, chunk_kib, procs, limit):
    import torch
    import bench
    from paper_2508_19263_b200 import binding as zc
    from paper_2508_19263_b200 import workloads as wl

    dev = torch.device("cuda", 0)
    fmt, specs = bench.workload_specs(workload)
    if workload.endswith("_static"):
        raise SystemExit("the *_static workloads share dictionaries between tensors: see tests/test_gpu_kv_dictionary.py")
    delta = "_delta" in workload                 # the XOR with the earlier checkpoint is what is coded
    frozen = workload.endswith("_delta_frozen")  # ... with a share of the rows left untouched
    if limit:
        specs = specs[:limit]
    chunk_bytes = chunk_kib * 1024
    tmp = tempfile.mkdtemp(prefix="zc_parity_", dir="/dev/shm" if os.path.isdir("/dev/shm") else None)
    t0 = time.time()
    n_bytes = n_cont = 0
    pending = {}
    try:
        with ProcessPoolExecutor(max_workers=procs, mp_context=mp.get_context("spawn")) as pool:
            def drain(block_until):
                while len(pending) > block_until:
                    done, _ = wait(list(pending), return_when=FIRST_COMPLETED)
                    for f in done:
                        name = pending.pop(f)
                        err = f.result()
                        if err:
                            raise SystemExit(f"{workload}: tensor {name}: {err}")

            group, group_bytes = [], 0
            def flush_group():
                nonlocal n_bytes, n_cont
                if not group:
                    return
                plans = [zc.plan(fmt, n, chunk_bytes) for _, _, n, _ in group]
                ins = [t for _, t, _, _ in group]
                bases = [b for _, _, _, b in group] if delta else None
                d_hist = torch.zeros((len(group), 2, 256), dtype=torch.int64, device=dev)
                zc.histogram_batch(zc.HistogramBatch(plans, ins, bases), d_hist)
                hists = d_hist.cpu().numpy().astype(np.uint64)
                cbs = zc.build_codebooks(plans, hists, zc.POLICY_AUTO)
                outs = [torch.empty(p.max_compressed_bytes, dtype=torch.uint8, device=dev) for p in plans]
                enc = zc.CompressBatch(plans, ins, outs, bases)
                enc.set_codebooks(cbs)
                ws = torch.empty(enc.workspace_bytes, dtype=torch.uint8, device=dev)
                sizes = zc.compress_batch(enc, ws)
                backs = [torch.empty(p.input_bytes, dtype=torch.uint8, device=dev) for p in plans]
                dws = torch.zeros(256, dtype=torch.uint8, device=dev)
                zc.decompress_batch(zc.DecompressBatch(plans, outs, sizes, backs, bases), dws)
                if zc.batch_status(dws) != (zc.OK, None):
                    raise SystemExit(f"{workload}: batched decoder status {zc.batch_status(dws)}")
                for i, (name, t, n, base) in enumerate(group):
                    if not torch.equal(backs[i], t[: plans[i].input_bytes]):
                        raise SystemExit(f"{workload}: tensor {name}: GPU round trip differs")
                    dp, cp = os.path.join(tmp, f"{name}.in.npy"), os.path.join(tmp, f"{name}.zc.npy")
                    coded = t if base is None else t ^ base
                    np.save(dp, coded[: plans[i].input_bytes].cpu().numpy())
                    np.save(cp, outs[i][: sizes[i]].cpu().numpy())
                    n_bytes += plans[i].input_bytes
                    n_cont += sizes[i]
                    drain(3 * procs)
                    pending[pool.submit(oracle_check, fmt, n, chunk_bytes, dp, cp, hists[i])] = name
                group.clear()

            for spec in specs:
                base = None
                if delta:
                    t, base, n = wl.checkpoint_pair(spec, dev, frozen_rows=wl.frozen_rows_of(spec) if frozen else 0.0)
                elif spec.name.startswith("kv."):
                    t, n = wl.kv_cache_tensor(fmt, spec.seed // 10, spec.seed % 10, dev)
                else:
                    t, n, _ = wl.make_weight(spec, fmt, dev)
                group.append((spec.name, t, n, base))
                group_bytes += t.numel() * (2 if delta else 1)
                if group_bytes >= (2 << 30):
                    flush_group()
                    group_bytes = 0
            flush_group()
            drain(0)
    finally:
        shutil.rmtree(tmp, ignore_errors=True)
    print(f"{workload}: {len(specs)} tensors, {n_bytes} bytes in, {n_cont} container bytes (ratio {n_cont / max(n_bytes, 1):.4f}), "
          f"chunks of {chunk_kib} KiB: histograms, containers and round trips identical to the oracle's "
          f"({procs} oracle processes, {time.time() - t0:.0f} s)")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", action="append", help="bench.py workload name; may be given several times")
    ap.add_argument("--chunk-kib", type=int, default=4)
    ap.add_argument("--procs", type=int, default=min(16, os.cpu_count() or 1))
    ap.add_argument("--limit", type=int, default=0, help="only the first N tensors of each workload")
    args = ap.parse_args()
    for w in args.workload or ["cfg2_bf16_llama8b"]:
        run(w, args.chunk_kib, args.procs, args.limit)


if __name__ == "__main__":
    main()
