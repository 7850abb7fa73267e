#!/usr/bin/env python
"""Benchmark of the walk + SGNS hot path on synthetic power-law graphs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One step = one mini-batch of the whole path: generate `batch_walks` random walks from the
CSR graph, expand them to (center, context) pairs with negative draws, and apply the SGNS
update to the embedding tables (lock-free mode for the large workloads).  The default
workload is the 50M-node DeepWalk configuration.  Prints ONE JSON line.

`value` is pair-updates/s with every input resident in HBM; `e2e` is the same metric with
the step's host inputs (start nodes, pinned memory) copied in and its result (loss, pair
count) copied out inside the timed region, through the same C-ABI calls.  `roofline` is
for the SGNS kernel (the dominant one); `walk` gives the walk sampler's own figures.
With --gpus N every rank runs an independent replica of the same workload on its own GPU
(the path has no exchange step); the value is the sum over ranks divided by the slowest
rank's time.

The default single-GPU run also carries `per_config`: short legs over the other named
workloads and the synchronous mode (device-resident timing only), each with its own roofline
block; --no-per-config leaves them out.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

METRIC = "sgns_pair_updates_per_s"
UNIT = "pair-updates/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="deepwalk_large")
    ap.add_argument("--scale", type=float, default=1.0, help="shrink the node count (testing)")
    ap.add_argument("--dim", type=int, default=None, choices=[32, 64, 128, 256],
                    help="embedding dimension instead of the workload's own (a sweep over the embedding "
                         "size, as in the paper's Fig. 11); named in config.dim")
    ap.add_argument("--batch-walks", type=int, default=1 << 20)
    ap.add_argument("--mode", default="hogwild_red",
                    choices=["hogwild", "hogwild_red", "deterministic", "momentum", "adam"],
                    help="hogwild_red: lock-free, increments added by reductions (default); "
                         "hogwild: lock-free with plain stores; deterministic: synchronous batches of 512 "
                         "walks; momentum / adam: synchronous with that optimizer")
    ap.add_argument("--variants", default="",
                    help="comma list of shrink (per-position window draw), subsample (frequent-node "
                         "sub-sampling, t = 1e-5), shuffle (keyed start-node order)")
    ap.add_argument("--table-dtype", default="f32", choices=["f32", "f16", "bf16"],
                    help="storage type of the embedding tables (arithmetic is fp32 either way)")
    ap.add_argument("--round", default="nearest", choices=["nearest", "stochastic"],
                    help="write-back rounding of 16-bit tables")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-sample-walks", type=int, default=16384)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the end-to-end leg (profiling runs)")
    ap.add_argument("--no-walk-index", action="store_true",
                    help="walk over the plain CSR (two random reads per transition)")
    ap.add_argument("--no-edge-set", action="store_true",
                    help="node2vec: membership in adj(prev) by binary search instead of the hashed edge set")
    ap.add_argument("--n2v-lanes", type=int, default=None,
                    help="node2vec kernel: 0 one lane per walk, flattened loop (default); 1, 2, 4, 8, 32: the "
                         "generic kernel with that many lanes per walk")
    ap.add_argument("--stage", default="all", choices=["all", "walks", "row-updates"],
                    help="'walks' times the walk sampler alone (no tables are allocated); 'row-updates' measures "
                         "the device's ceiling for random row read-modify-write (no workload is built)")
    ap.add_argument("--no-per-config", action="store_true",
                    help="skip the short legs over the other workloads that the default run adds")
    ap.add_argument("--cpu-workers", type=int, default=0,
                    help="processes of the all-cores oracle leg (0: one per usable core, at most 64)")
    return ap.parse_args()


# ---------------------------------------------------------------------------- helpers
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "200", "-i", str(self.index)], stdout=f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        try:
            rows = [l.split(",") for l in open(self.path).read().strip().splitlines() if l.strip()]
            os.unlink(self.path)
            sm = [float(r[0]) for r in rows]
            out["sm_mhz"] = statistics.median(sm) if sm else None
            out["sm_max_mhz"] = float(rows[0][1]) if rows else None
            out["power_w_max"] = max(float(r[2]) for r in rows) if rows else None
            names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
            out["reasons"] = [n for k, n in enumerate(names)
                              if any("Active" in r[3 + k] and "Not" not in r[3 + k] for r in rows)]
            out["samples"] = len(rows)
        except Exception as e:          # clock sampling must never break the benchmark
            out["error"] = str(e)
        return out


def measured_peak_gbs():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


NOMINAL_HBM_GBS = 8000.0      # the device's nominal HBM3e bandwidth, for context


def recorded_traffic(kernel, workload):
    """DRAM bytes per pair (or per transition) of `kernel` taken from the ncu summary under
    profiles/, with the note that says where they were captured, or (None, None) when there is
    none or the kernel's source has changed since the capture.  The summary records the sha256 of
    the part of the source file that holds the kernel: everything before the line `upto`."""
    import hashlib
    import re
    f = ROOT / "profiles" / f"{kernel}__{workload}.md"
    if not f.exists():
        return None, None
    text = f.read_text()
    m = re.search(r"dram_bytes_per_unit\s*=\s*([0-9.eE+-]+)", text)
    h = re.search(r"source\s*=\s*(\S+)\s+upto\s*=\s*\"([^\"]+)\"\s+sha256\s*=\s*([0-9a-f]{64})", text)
    note = re.search(r"traffic_note\s*=\s*(.+)", text)
    if not m or not h:
        return None, None
    src = ROOT / h.group(1)
    if not src.exists():
        return None, None
    body = src.read_text()
    cut = body.find(h.group(2))
    if cut < 0 or hashlib.sha256(body[:cut].encode()).hexdigest() != h.group(3):
        return None, None
    return float(m.group(1)), note.group(1).strip() if note else None


def algorithmic_bytes(pairs, positions, dim, n_neg, elem=4):
    """Row traffic the update must move: per pair 1+K output rows read and written plus K
    alias entries; per center position one input row read and written plus its walk entry.
    elem = bytes per stored table value."""
    return pairs * ((1 + n_neg) * 2 * elem * dim + 8 * n_neg) + positions * (2 * elem * dim + 4)


def walk_bytes(steps, offsets64, indexed=False):
    """Payload of a walk transition: two offsets and one column (or one 16-byte index record),
    plus the stored entry."""
    return steps * ((16 if indexed else (16 if offsets64 else 8) + 4) + 4)


def walk_granule_bytes(steps, indexed=False):
    """DRAM cannot move less than a 64-byte granule per isolated random read (measured: the
    64-byte fetch hint is the smallest the L2 honours): one granule per record, or one for the
    offset pair and one for the column, plus the 4 bytes stored."""
    return steps * ((64 if indexed else 128) + 4)


def build_inputs(wl, scale, device):
    from paper_2407_15452_b200 import binding as B
    t0 = time.time()
    g = wl.make_graph(device=device, scale=scale)
    deg = g.degrees()
    info = {"n_nodes": g.n_nodes, "n_edges": g.n_edges, "max_degree": int(deg.max()),
            "frac_isolated": float((deg == 0).double().mean()), "graph_s": round(time.time() - t0, 1)}
    t0 = time.time()
    table = B.gs_build_alias(deg.cpu().numpy().astype(np.float64), 0.75)
    info["alias_s"] = round(time.time() - t0, 1)
    return g, table, info


# ---------------------------------------------------------------------------- CPU oracle leg
def oracle_sample(wl, off, col, table, n_walks, base, seed):
    """Times the CPU oracle on `n_walks` walks of the workload: walks, pair/negative expansion,
    sequential SGNS on the touched rows.  Returns (pairs, steps, seconds by stage)."""
    from oracle import gs_oracle as O
    thr = (table & np.uint64(0xFFFFFFFF)).astype(np.uint32)
    alias = (table >> np.uint64(32)).astype(np.int32)
    t0 = time.perf_counter()
    if wl.walk_kind == "uniform":
        walks, steps = O.uniform_walks(off, col, None, n_walks, base, wl.walk_len, seed)
    else:
        walks, steps, _ = O.node2vec_walks(off, col, None, n_walks, base, wl.walk_len, seed, wl.p, wl.q)
    t1 = time.perf_counter()
    c, o, ng, pairs = O.expand_lists(walks, base, wl.window, wl.n_neg, thr, alias, seed,
                                     forward_only=wl.forward_only)
    t2 = time.perf_counter()
    # input data handling (not timed): renumber touched rows, materialise their start values
    allv = np.concatenate([c, o, ng.ravel()])
    ids = np.unique(allv[allv >= 0])
    remap = lambda a: np.where(a >= 0, np.searchsorted(ids, np.maximum(a, 0)), -1).astype(np.int32)
    cc, oo, nn = remap(c), remap(o), remap(ng)
    U = O.init_rows(ids, wl.dim, seed)
    V = np.zeros_like(U)
    t3 = time.perf_counter()
    O.sgns_seq_from_lists(U, V, cc, oo, nn, 2 * wl.window, wl.lr0)
    t4 = time.perf_counter()
    return pairs, steps, {"walk_s": t1 - t0, "expand_s": t2 - t1, "sgns_s": t4 - t3}


def _oracle_worker(job):
    """One process of the all-cores oracle leg: maps the shared inputs and runs the oracle, as it
    stands, on its own range of walk ids (its own copy of the touched rows).  Returns
    (pairs, steps, seconds of oracle work)."""
    folder, wl_name, n_walks, base, seed, start_at = job
    from paper_2407_15452_b200.workloads import WORKLOADS
    wl = WORKLOADS[wl_name]
    off = np.load(os.path.join(folder, "off.npy"), mmap_mode="r")
    col = np.load(os.path.join(folder, "col.npy"), mmap_mode="r")
    table = np.load(os.path.join(folder, "alias.npy"), mmap_mode="r")
    n_nodes = len(off) - 1
    # the sample's own part of the alias table is small next to the CSR: read it whole
    table = np.ascontiguousarray(table)
    oracle_sample(wl, off, col, table, 8, base, seed)            # loads the library, touches pages
    while time.time() < start_at:                                 # all processes start together
        time.sleep(0.005)
    p, st, t = oracle_sample(wl, off, col, table, n_walks, base, seed)
    return p, st, t["walk_s"] + t["expand_s"] + t["sgns_s"], n_nodes


def oracle_all_cores(wl, off, col, table, seed, workers, walks_each):
    """The oracle on all host cores: `workers` processes (spawned, so that none inherits a CUDA
    context), each running the single-threaded oracle on a disjoint range of walk ids with its own
    copy of the rows it touches.  Rate = pairs of all processes / slowest process."""
    import multiprocessing as mp
    import shutil
    usable = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    if workers <= 0:
        workers = min(usable, 64)
    root = "/dev/shm" if os.path.isdir("/dev/shm") and os.access("/dev/shm", os.W_OK) else None
    folder = tempfile.mkdtemp(prefix="gs_oracle_", dir=root)
    try:
        np.save(os.path.join(folder, "off.npy"), off)
        np.save(os.path.join(folder, "col.npy"), col)
        np.save(os.path.join(folder, "alias.npy"), table)
        start_at = time.time() + 3.0 + 0.1 * workers
        jobs = [(folder, wl.name, walks_each, (1 << 20) + k * walks_each, seed, start_at) for k in range(workers)]
        with mp.get_context("spawn").Pool(workers) as pool:
            res = pool.map(_oracle_worker, jobs, chunksize=1)
    finally:
        shutil.rmtree(folder, ignore_errors=True)
    pairs = sum(r[0] for r in res)
    steps = sum(r[1] for r in res)
    slowest = max(r[2] for r in res)
    return {"value": pairs / slowest, "unit": UNIT, "cores": workers, "host_cores": usable,
            "kind": "oracle, one single-threaded process per core on disjoint walk-id ranges",
            "sample": f"{workers} x {walks_each} walks ({slowest:.1f} s for the slowest process)",
            "walk_steps": steps}


def run_reference(args, wl):
    """--impl reference: the CPU oracle, as it stands, on the host cores.  Nothing of the CUDA
    library is loaded: the alias table comes from the oracle's own builder."""
    import torch
    from oracle import gs_oracle as O
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    device = "cuda" if torch.cuda.is_available() else "cpu"
    scale = args.scale if device == "cuda" else min(args.scale, 0.02)
    t0 = time.time()
    g = wl.make_graph(device=device, scale=scale)
    deg = g.degrees()
    info = {"n_nodes": g.n_nodes, "n_edges": g.n_edges, "max_degree": int(deg.max()),
            "frac_isolated": float((deg == 0).double().mean()), "graph_s": round(time.time() - t0, 1)}
    t0 = time.time()
    thr, alias = O.build_alias(deg.cpu().numpy().astype(np.float64), 0.75)
    table = (alias.astype(np.uint64) << np.uint64(32)) | thr.astype(np.uint64)
    info["alias_s"] = round(time.time() - t0, 1)
    off = g.offsets.cpu().numpy().astype(np.int64)
    col = g.cols.cpu().numpy()
    del g, deg, thr, alias
    n = min(max(args.cpu_sample_walks // 8, 1), 1024)
    for s in range(args.warmup):
        oracle_sample(wl, off, col, table, n, s * n, wl.graph_seed)
    pairs = steps = 0
    secs = 0.0
    for s in range(args.steps):
        p, st, t = oracle_sample(wl, off, col, table, n, (args.warmup + s) * n, wl.graph_seed)
        pairs += p
        steps += st
        secs += t["walk_s"] + t["expand_s"] + t["sgns_s"]
    value = pairs / secs
    sample = f"{n} walks per step (walks + pair/negative expansion + sequential SGNS on touched rows)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "gpu_launches": 0,
        "config": {"workload": wl.name, "scale": scale, **info},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def walk_kernel_name(wl, indexed):
    if wl.walk_kind != "uniform":
        return "node2vec_flat_kernel"
    return "uniform_walk_index_kernel" if indexed else "uniform_walk_vec_kernel"


def sync_step_launches(n_nodes, extra=0):
    """Kernels of one synchronous batch: walks; targets and three per radix pass of at most 8 bits
    over keys below 2 n_nodes (the table-independent part); coefficients, apply of the output
    rows, and the last launch (input rows, cut runs, sums)."""
    passes = ((2 * n_nodes).bit_length() + 7) // 8
    return 1 + 1 + 3 * passes + 1 + 2 + extra


def parse_variants(args):
    v = {x for x in args.variants.split(",") if x}
    bad = v - {"shrink", "subsample", "shuffle"}
    if bad:
        raise SystemExit(f"unknown variant(s): {sorted(bad)}")
    return v


def keep_thresholds_device(g, dev, t=1e-5):
    """Sub-sampling thresholds from the degrees (host call of the library), uploaded."""
    import torch
    from paper_2407_15452_b200 import binding as B
    thr = B.gs_build_keep_thresholds(g.degrees().cpu().numpy().astype(np.float64), t)
    return torch.from_numpy(thr.view(np.int32)).to(dev)


def probe_random_reads(n_records, n_reads, dev):
    """Independent random 16-byte reads per second over a buffer of n_records records, measured by
    the benchmark's own probe library (libbench_probe.so, built from bench_probe.cu)."""
    import ctypes
    import torch
    so = ROOT / "libbench_probe.so"
    if not so.exists():
        return None
    lib = ctypes.CDLL(str(so))
    buf = torch.zeros(n_records * 4, dtype=torch.int32, device=dev)
    done, ms = ctypes.c_int64(0), ctypes.c_float(0.0)
    rc = lib.bench_probe_random_reads(ctypes.c_void_p(buf.data_ptr()), ctypes.c_int64(n_records),
                                      ctypes.c_int64(n_reads), ctypes.byref(done), ctypes.byref(ms),
                                      ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    del buf
    if rc != 0 or ms.value <= 0:
        return None
    return done.value / (ms.value * 1e-3)


def run_row_update_probe(args):
    """The ceiling of the update kernels' access pattern, measured with the benchmark's own probe
    library: rows of 256 bytes (dim 128 in a 16-bit format) and 512 bytes (dim 128 in fp32) of a 4 GB
    table visited at random, each read and written back, nothing computed.  One JSON line."""
    import ctypes
    import torch
    so = ROOT / "libbench_probe.so"
    if not so.exists():
        raise SystemExit("libbench_probe.so is missing: run python -m paper_2407_15452_b200.build")
    lib = ctypes.CDLL(str(so))
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    table_bytes, n_visits = 4 << 30, 1 << 23
    table = torch.zeros(table_bytes // 4, dtype=torch.int32, device=dev)
    peak, peak_kind = measured_peak_gbs()
    rows_out = []
    for row_bytes in (256, 512):
        n_rows = table_bytes // row_bytes
        gen = torch.Generator(device=dev)
        gen.manual_seed(12345)
        ids = torch.randint(0, n_rows, (n_visits,), dtype=torch.int32, device=dev, generator=gen)
        for write in (0, 1):
            best = None
            for in_flight in (3, 6):
                for bps in (4, 8, 16):
                    ms = ctypes.c_float(0.0)
                    rc = lib.bench_probe_row_updates(
                        ctypes.c_void_p(table.data_ptr()), ctypes.c_int64(n_rows), ctypes.c_int32(row_bytes),
                        ctypes.c_void_p(ids.data_ptr()), ctypes.c_int64(n_visits), ctypes.c_int32(in_flight),
                        ctypes.c_int32(bps), ctypes.c_int32(write), ctypes.byref(ms),
                        ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
                    if rc != 0 or ms.value <= 0:
                        raise SystemExit(f"bench_probe_row_updates failed with CUDA error {rc}")
                    gbs = n_visits * row_bytes * (2 if write else 1) / (ms.value * 1e-3) / 1e9
                    if best is None or gbs > best["gbs"]:
                        best = {"row_bytes": row_bytes, "write_back": bool(write), "gbs": gbs,
                                "rows_per_s": n_visits / (ms.value * 1e-3), "accesses_in_flight": in_flight,
                                "blocks_per_sm": bps, "frac_of_copy_rate": gbs / peak}
            rows_out.append(best)
    print(json.dumps({"metric": "row_update_ceiling", "unit": "GB/s", "n_gpus": 1, "data": "synthetic",
                      "config": {"stage": "row-updates", "table_bytes": table_bytes, "visits": n_visits,
                                 "note": "best over 3 or 6 accesses in flight per warp and 4, 8, 16 blocks of "
                                         "4 warps per SM; one warm-up and one timed launch each"},
                      "peak": peak, "peak_kind": f"of {peak_kind}", "results": rows_out}))


# ---------------------------------------------------------------------------- walk sampler alone
def run_walks_only(args, wl, g, G, info, dev):
    """Times gs_random_walks / gs_node2vec_walks alone on batches of the workload (1 GPU)."""
    import torch
    from paper_2407_15452_b200 import binding as B
    n = g.n_nodes
    total_walks = n * wl.walks_per_node
    bw = min(args.batch_walks, total_walks)
    nb_total = (total_walks + bw - 1) // bw
    out = torch.empty((bw, wl.walk_len), dtype=torch.int32, device=dev)
    steps = torch.zeros(1, dtype=torch.int64, device=dev)
    variants = parse_variants(args)
    starts = torch.empty(bw, dtype=torch.int32, device=dev) if "shuffle" in variants else None
    keep_thr = keep_thresholds_device(g, dev) if "subsample" in variants else None
    kept = torch.zeros(1, dtype=torch.int64, device=dev)

    def run(b):
        base = (b % nb_total) * bw
        cnt = min(bw, total_walks - base)
        if starts is not None:
            B.gs_shuffled_starts(n, wl.graph_seed, 0, base, cnt, dev, out=starts)
        if wl.walk_kind == "uniform":
            B.gs_random_walks(G, starts, cnt, base, wl.walk_len, wl.graph_seed, out=out, steps=steps)
        else:
            B.gs_node2vec_walks(G, starts, cnt, base, wl.walk_len, wl.graph_seed, wl.p, wl.q, out=out,
                                steps=steps)
        if keep_thr is not None:
            B.gs_subsample_walks(out[:cnt], base, keep_thr, wl.graph_seed, out=out[:cnt], kept=kept)

    for s in range(args.warmup):
        run(s)
    torch.cuda.synchronize()
    steps.zero_()
    kept.zero_()
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for s in range(args.steps):
        run(args.warmup + s)
    ev1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1)
    st = int(steps.item())
    peak, peak_kind = measured_peak_gbs()
    indexed = "walk_index_bytes" in info
    payload = walk_bytes(st, wl.offsets64, indexed) / (ms * 1e-3) / 1e9
    granule = walk_granule_bytes(st, indexed) / (ms * 1e-3) / 1e9
    # ceiling of one isolated random read per transition, measured in this run on a buffer of the
    # walk index's size (16 bytes per CSR entry)
    read_rate = probe_random_reads(g.n_edges, 1 << 28, dev) if indexed else None
    print(json.dumps({
        "metric": "walk_steps_per_s", "value": st / (ms * 1e-3), "unit": "walk-steps/s", "n_gpus": 1,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32",
        "data": "synthetic", "gpu_launches": args.steps * (1 + len(variants & {"shuffle", "subsample"})),
        "clocks": clocks,
        "config": {"workload": wl.name, "stage": "walks", "batch_walks": bw, "walk_kind": wl.walk_kind,
                   "walk_len": wl.walk_len, "scale": args.scale, "variants": sorted(variants),
                   "kept_entries": int(kept.item()) if keep_thr is not None else None, **info},
        "roofline": {"bound": "hbm", "kernel": walk_kernel_name(wl, indexed),
                     "achieved": payload, "peak": peak, "unit": "GB/s", "frac": payload / peak,
                     "peak_kind": f"of {peak_kind}", "traffic": None,
                     "granule_gbs": granule, "granule_frac": granule / peak,
                     "random_reads_per_s": read_rate,
                     "frac_of_random_read_rate": st / (ms * 1e-3) / read_rate if read_rate else None},
    }))


# ---------------------------------------------------------------------------- momentum step
def run_momentum(args, wl, g, G, alias, w_in, w_out, info, dev):
    """Times the epoch driver with the momentum (or, --mode adam, Adam) step on batches of 512 walks
    (synchronous; momentum 0.9 as in the paper's production run).  1 GPU."""
    import torch
    from paper_2407_15452_b200 import binding as B
    n = g.n_nodes
    bw = min(args.batch_walks, 512)
    total_walks = n * wl.walks_per_node
    nb_total = (total_walks + bw - 1) // bw
    adam = args.mode == "adam"
    m_in, m_out = torch.zeros_like(w_in), torch.zeros_like(w_out)
    if adam:
        v_in, v_out = torch.zeros_like(w_in), torch.zeros_like(w_out)
    else:
        last_in = torch.zeros(n, dtype=torch.int32, device=dev)
        last_out = torch.zeros_like(last_in)
    mu = 0.9
    seed, lr = wl.graph_seed, wl.lr0 * (1.0 - mu)      # same effective step lr / (1 - mu) as the plain runs
    if adam:
        lr = 0.001                                     # Adam's usual step size
    kind = B.GS_WALK_UNIFORM if wl.walk_kind == "uniform" else B.GS_WALK_NODE2VEC
    kw = dict(walks_per_node=wl.walks_per_node, walk_len=wl.walk_len, window=wl.window, n_neg=wl.n_neg,
              lr0=lr, batch_walks=bw, seed=seed, mode=B.GS_DETERMINISTIC, walk_kind=kind, p=wl.p, q=wl.q,
              momentum=mu, m_in=m_in, m_out=m_out)
    if adam:
        kw.update(optimizer=B.GS_OPT_ADAM, beta2=0.999, eps=1e-8, v_in=v_in, v_out=v_out)
    else:
        kw.update(optimizer=B.GS_OPT_MOMENTUM, last_in=last_in, last_out=last_out)
    # the epoch driver runs the optimizer step per batch; one call covers the K timed batches
    assert args.warmup + args.steps <= nb_total
    B.gs_sgns_epoch(G, alias, w_in, w_out, first_batch=0, num_batches=args.warmup, **kw)
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    r = B.gs_sgns_epoch(G, alias, w_in, w_out, first_batch=args.warmup, num_batches=args.steps, **kw)
    ev1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1)
    pairs = r.pairs
    loss = torch.tensor([r.loss_sum])
    peak, peak_kind = measured_peak_gbs()
    # per pair and target: the embedding row and its momentum row (Adam: both moment rows), each
    # read and written once
    model = pairs * (1 + wl.n_neg) * (6 if adam else 4) * wl.dim * 4
    gbs = model / (ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": METRIC, "value": pairs / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "gpu_launches": sync_step_launches(n, 0 if adam else 1) * args.steps,   # momentum: + catch-up
        "clocks": clocks, "mean_loss": loss.item() / max(pairs, 1),
        "config": {"workload": wl.name, "mode": args.mode, "momentum": mu, "lr": lr, "batch_walks": bw,
                   "walk_len": wl.walk_len, "window": wl.window, "n_neg": wl.n_neg, "dim": wl.dim,
                   "scale": args.scale, **info},
        "roofline": {"bound": "hbm", "kernel": "adam step (coefficients, sort, apply)" if adam else
                     "momentum step (keys, sort, catch-up, coefficients, apply)",
                     "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                     "peak_kind": f"of {peak_kind}", "traffic": None,
                     "bytes_model": "per pair and target: row and moment row(s), read + written"},
    }))


# ---------------------------------------------------------------------------- our arm
def fractions(gbs, peak):
    """The same rate against the measured copy bandwidth and against the nominal figure."""
    return {"frac": gbs / peak, "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS}


def run_leg(args, wl, dev, rank, world, local, with_e2e, with_cpu):
    """Builds the inputs of `wl`, times the path as `args` says and returns the result line as a
    dict (rank 0; None elsewhere).  Frees everything it allocated on the device."""
    import torch
    import torch.distributed as dist
    from paper_2407_15452_b200 import binding as B
    from paper_2407_15452_b200 import replicas

    g, table, info = build_inputs(wl, args.scale, dev)
    n = g.n_nodes
    flags = B.GS_VALIDATE | B.GS_REQUIRE_SORTED
    if not args.no_walk_index:
        flags |= B.GS_BUILD_WALK_INDEX                  # 16 B per CSR entry, one read per transition
        info["walk_index_bytes"] = 16 * g.n_edges
    if wl.walk_kind != "uniform" and not args.no_edge_set:
        info["edge_set"] = True
        flags |= B.GS_BUILD_EDGE_SET                    # hashed "is x a neighbour of prev" for node2vec
    G = B.gs_graph_load_csr(g.offsets, g.cols, flags)
    if args.n2v_lanes is not None:
        B.gs_tune_node2vec_group(args.n2v_lanes)
    if args.stage == "walks":
        return run_walks_only(args, wl, g, G, info, dev)
    alias = torch.from_numpy(table.view(np.int64)).to(dev)
    f16 = args.table_dtype != "f32"                    # a 16-bit storage format
    tdt = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}[args.table_dtype]
    w_in = torch.empty((n, wl.dim), dtype=tdt, device=dev)
    w_out = torch.empty_like(w_in)
    seed = wl.graph_seed
    {"f32": B.gs_init_embeddings, "f16": B.gs_init_embeddings_f16,
     "bf16": B.gs_init_embeddings_bf16}[args.table_dtype](w_in, w_out, seed)
    step_fn = {"f32": B.gs_sgns_step, "f16": B.gs_sgns_step_f16, "bf16": B.gs_sgns_step_bf16}[args.table_dtype]
    if args.mode in ("momentum", "adam"):
        return run_momentum(args, wl, g, G, alias, w_in, w_out, info, dev)
    mode_name = args.mode
    if f16 and mode_name == "hogwild_red" and args.round == "stochastic":
        mode_name = "hogwild"                          # the reduction unit rounds to nearest only
    mode = {"hogwild": B.GS_HOGWILD, "hogwild_red": B.GS_HOGWILD_RED,
            "deterministic": B.GS_DETERMINISTIC}[mode_name]
    if wl.forward_only:
        mode |= B.GS_PAIRS_FORWARD_ONLY
    variants = parse_variants(args)
    if "shrink" in variants:
        mode |= B.GS_WINDOW_SHRINK
    if args.round == "stochastic":
        if not f16:
            raise SystemExit("--round stochastic needs --table-dtype f16 or bf16")
        mode |= B.GS_ROUND_STOCHASTIC
    keep_thr = keep_thresholds_device(g, dev) if "subsample" in variants else None
    kind = B.GS_WALK_UNIFORM if wl.walk_kind == "uniform" else B.GS_WALK_NODE2VEC
    total_walks = n * wl.walks_per_node
    bw = min(args.batch_walks, total_walks)
    if (mode & 0xFF) == B.GS_DETERMINISTIC:
        bw = min(bw, 512)
    nb_total = (total_walks + bw - 1) // bw
    lr_schedule = B.GS_LR_LINEAR if wl.lr_schedule == "linear" else B.GS_LR_CONSTANT
    ekw = dict(walks_per_node=wl.walks_per_node, walk_len=wl.walk_len, window=wl.window,
               n_neg=wl.n_neg, lr0=wl.lr0, batch_walks=bw, seed=seed, mode=mode, walk_kind=kind,
               p=wl.p, q=wl.q, keep_thr=keep_thr, shuffle_epoch=0 if "shuffle" in variants else None,
               lr_schedule=lr_schedule)
    n_steps = min(args.steps, max(nb_total - args.warmup, 1))   # a small workload has fewer batches

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def batch_of(step):                                # replicas walk disjoint parts of the epoch
        return replicas.batch_of(step, rank, world, nb_total)

    # ---- device-resident timing -------------------------------------------------------
    # warm-up: one call per batch, so the walk kernel runs alone here (inside a multi-batch call it
    # shares the GPU with the update of the previous batch); its own figures are taken from these
    warm = [B.gs_sgns_epoch(G, alias, w_in, w_out, first_batch=batch_of(s), num_batches=1, **ekw)
            for s in range(args.warmup)]
    warm = warm[1:] if len(warm) > 1 else warm
    sampler = ClockSampler(local)
    barrier()
    if rank == 0:
        sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    pairs = steps = walks_done = 0
    loss = 0.0
    ms_walk = ms_sgns = 0.0
    ev0.record()
    # One replica takes consecutive mini-batches: the K timed steps are ONE call of the epoch
    # driver over K batches, as a user runs it (walk generation of batch b+1 then overlaps the
    # update of batch b).  Several replicas interleave their batches, so they call per step.
    one_call = world == 1 and args.warmup + n_steps <= nb_total
    calls = [(args.warmup, n_steps)] if one_call else \
            [(batch_of(args.warmup + s), 1) for s in range(n_steps)]
    for b, nb in calls:
        r = B.gs_sgns_epoch(G, alias, w_in, w_out, first_batch=b, num_batches=nb, **ekw)
        pairs += r.pairs
        steps += r.steps
        loss += r.loss_sum
        ms_walk += r.ms_walk
        ms_sgns += r.ms_sgns
        walks_done += sum(min(bw, total_walks - x * bw) for x in range(b, b + nb))
    ev1.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms = ev0.elapsed_time(ev1)

    # ---- end to end: host inputs in, result out, same C-ABI calls ---------------------------
    e2e_pairs, e2e_s = 0, float("nan")
    if with_e2e:
        h_starts = torch.empty(bw, dtype=torch.int32).pin_memory()
        d_starts = torch.empty(bw, dtype=torch.int32, device=dev)
        d_walks = torch.empty((bw, wl.walk_len), dtype=torch.int32, device=dev)
        d_res = torch.zeros(2, dtype=torch.float64, device=dev)   # [loss, pair count as int64 bits]
        d_loss = d_res[0:1]
        d_cnt = d_res[1:2].view(torch.int64)
        h_res = torch.zeros(2, dtype=torch.float64).pin_memory()

        def e2e_step(step):
            b = batch_of(step)
            base = b * bw
            cnt = min(bw, total_walks - base)
            h_starts[:cnt] = (torch.arange(base, base + cnt, dtype=torch.int64) % n).to(torch.int32)
            d_starts[:cnt].copy_(h_starts[:cnt], non_blocking=True)
            d_res.zero_()
            if kind == B.GS_WALK_UNIFORM:
                B.gs_random_walks(G, d_starts, cnt, base, wl.walk_len, seed, out=d_walks)
            else:
                B.gs_node2vec_walks(G, d_starts, cnt, base, wl.walk_len, seed, wl.p, wl.q, out=d_walks)
            if keep_thr is not None:
                B.gs_subsample_walks(d_walks[:cnt], base, keep_thr, seed, out=d_walks[:cnt])
            step_fn(w_in, w_out, d_walks[:cnt], base, wl.window, wl.n_neg, alias, wl.lr0,
                    seed, mode, d_loss, d_cnt)
            h_res.copy_(d_res, non_blocking=True)
            torch.cuda.synchronize()
            return int(h_res[1:2].view(torch.int64).item())

        for s in range(min(args.warmup, 2)):
            e2e_step(args.warmup + n_steps + s)
        barrier()
        t0 = time.perf_counter()
        for s in range(n_steps):
            e2e_pairs += e2e_step(args.warmup + n_steps + 2 + s)
        barrier()
        e2e_s = time.perf_counter() - t0

    # ---- max over ranks, sums over ranks ------------------------------------------------------
    (ms, e2e_s), (pairs_all, steps_all, e2e_pairs_all) = replicas.reduce_timing(
        [ms, e2e_s], [pairs, steps, e2e_pairs], device=dev)

    out = None
    if rank == 0:
        peak, peak_kind = measured_peak_gbs()
        launches = n_steps                                        # SGNS launches on this rank
        positions = steps + walks_done                            # walk entries = center positions
        sgns_bytes = algorithmic_bytes(pairs, positions, wl.dim, wl.n_neg, 2 if f16 else 4) / launches
        lock_free = (mode & 0xFF) != B.GS_DETERMINISTIC
        # lock-free: the update kernel's own time.  Synchronous: the whole step, because its kernels
        # run on two streams (targets and sort of the next batch beside the update of this one)
        sgns_ms = ms_sgns / launches if lock_free else ms / launches
        achieved = sgns_bytes / (sgns_ms * 1e-3) / 1e9
        indexed = "walk_index_bytes" in info
        if one_call and warm:                          # walk kernel alone: the warm-up calls
            w_steps, w_ms, w_n = sum(r.steps for r in warm), sum(r.ms_walk for r in warm), len(warm)
        else:
            w_steps, w_ms, w_n = steps, ms_walk, launches
        wbytes = walk_bytes(w_steps, wl.offsets64, indexed) / w_n
        gbytes = walk_granule_bytes(w_steps, indexed) / w_n
        walk_ms = w_ms / w_n
        per_pair, traffic_note = recorded_traffic("sgns_hogwild_kernel", wl.name) \
            if mode_name == "hogwild_red" and not f16 else (None, None)
        traffic = per_pair * pairs / launches if per_pair else None
        payload_gbs = wbytes / (walk_ms * 1e-3) / 1e9
        granule_gbs = gbytes / (walk_ms * 1e-3) / 1e9
        out = {
            "metric": METRIC, "value": pairs_all / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": n_steps, "warmup": args.warmup, "ms_per_step": ms / n_steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": wl.name, "mode": mode_name, "table_dtype": args.table_dtype,
                       "round": args.round if f16 else None, "batch_walks": bw,
                       "walk_kind": wl.walk_kind, "walk_len": wl.walk_len, "window": wl.window,
                       "n_neg": wl.n_neg, "dim": wl.dim, "scale": args.scale, "variants": sorted(variants),
                       "l2": "tables (2 x n x dim x 4 B) and CSR far exceed the 126 MB L2; no flush"
                             if 2 * n * wl.dim * (2 if f16 else 4) > (1 << 30) else
                             "every step takes a new batch of walks; tables of this workload are "
                             "smaller than 1 GB, rows may stay in the 126 MB L2 between steps",
                       "timed_region": "one gs_sgns_epoch call over the K batches" if one_call else
                                       "one gs_sgns_epoch call per batch",
                       "multi_gpu": "replicas only", **info},
            "gpu_launches": ((2 if lock_free else sync_step_launches(n))
                             + len(variants & {"shuffle", "subsample"})) * n_steps,
            "mean_loss": loss / max(pairs, 1),
            "walk_steps_per_s": steps_all / (ms * 1e-3),
            "clocks": clocks,
            "roofline": {"bound": "hbm",
                         "kernel": "sgns_hogwild_kernel" if lock_free else "synchronous step (coefficients, sort, apply)",
                         "achieved": achieved, "peak": peak, "unit": "GB/s", **fractions(achieved, peak),
                         "peak_kind": f"of {peak_kind}", "traffic": traffic, "traffic_note": traffic_note,
                         "ms_per_launch": sgns_ms, "pair_updates_per_s": pairs / (sgns_ms * launches * 1e-3),
                         "ms_update_stream": ms_sgns / launches},
            "walk": {"kernel": walk_kernel_name(wl, indexed),
                     "walk_steps_per_s_kernel": w_steps / (w_ms * 1e-3), "ms_per_launch": walk_ms,
                     "payload_gbs": payload_gbs, "payload_frac": payload_gbs / peak,
                     "payload_frac_of_nominal_8TBs": payload_gbs / NOMINAL_HBM_GBS,
                     "granule_gbs": granule_gbs, "granule_frac": granule_gbs / peak,
                     "granule_frac_of_nominal_8TBs": granule_gbs / NOMINAL_HBM_GBS,
                     "note": "payload = CSR bytes read + entries stored (the stated metric); granule "
                             "counts the 64 bytes DRAM moves per isolated read (supplementary)"},
        }
        if with_e2e:
            out["e2e"] = {"value": e2e_pairs_all / e2e_s, "unit": UNIT,
                          "h2d_bytes_per_step": 4 * bw, "d2h_bytes_per_step": 16}
        if with_cpu and world == 1:
            off = g.offsets.cpu().numpy().astype(np.int64)
            col = g.cols.cpu().numpy()
            p, st, t = oracle_sample(wl, off, col, table, args.cpu_sample_walks, 0, seed)
            tot = t["walk_s"] + t["expand_s"] + t["sgns_s"]
            out["cpu_baseline"] = {
                "value": p / tot, "unit": UNIT, "cores": 1, "kind": "oracle",
                "sample": f"first {args.cpu_sample_walks} walks of the workload: walks, pair/negative "
                          f"expansion, sequential SGNS on the touched rows ({tot:.1f} s)",
                "walk_steps_per_s": st / t["walk_s"], "sgns_pair_updates_per_s": p / t["sgns_s"]}
            try:
                out["cpu_baseline"]["all_cores"] = oracle_all_cores(wl, off, col, table, seed,
                                                                    args.cpu_workers, 1024)
            except Exception as e:                       # the single-core figure stands on its own
                out["cpu_baseline"]["all_cores"] = {"unavailable": f"{type(e).__name__}: {e}"}
    G.close()
    del w_in, w_out, alias, g, G
    B.gs_release_workspace()
    torch.cuda.empty_cache()
    return out


# The default run's short legs: (workload, mode, steps, warm-up, table type).  The synchronous mode
# takes batches of 512 walks, so its legs run a few hundred steps inside one call of the epoch
# driver; the tiny workload is its whole epoch (20 batches).  The last leg is the headline workload
# with half-precision tables (the storage type of the paper's production run, Section 4.2).
PER_CONFIG_LEGS = [
    ("tiny_deepwalk", "deterministic", 17, 3, "f32"),
    ("deepwalk_medium", "deterministic", 300, 5, "f32"),
    ("deepwalk_medium", "hogwild_red", 8, 3, "f32"),
    ("node2vec_4m", "hogwild_red", 6, 3, "f32"),
    ("rmat_billion", "hogwild_red", 10, 3, "f32"),
    ("deepwalk_large", "hogwild_red", 8, 3, "f16"),
]


def run_ours(args, wl):
    import argparse
    import torch
    import torch.distributed as dist
    from paper_2407_15452_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    B.lib()                                            # fail loudly if the library is missing

    plain = (args.workload == "deepwalk_large" and args.mode == "hogwild_red" and args.stage == "all"
             and args.table_dtype == "f32" and not args.variants and args.scale == 1.0 and args.dim is None)
    out = run_leg(args, wl, dev, rank, world, local, with_e2e=not args.no_e2e,
                  with_cpu=not args.no_cpu_baseline)
    if out is not None and plain and world == 1 and not args.no_per_config:
        legs = {}
        for name, mode, steps, warmup, tdt in PER_CONFIG_LEGS:
            from paper_2407_15452_b200.workloads import WORKLOADS
            largs = argparse.Namespace(**{**vars(args), "workload": name, "mode": mode, "steps": steps,
                                          "warmup": warmup, "batch_walks": 1 << 20, "table_dtype": tdt})
            t0 = time.time()
            r = run_leg(largs, WORKLOADS[name], dev, rank, world, local, with_e2e=False, with_cpu=False)
            legs[f"{name}/{mode}" + ("" if tdt == "f32" else f"/{tdt}")] = {
                "pair_updates_per_s": r["value"], "walk_steps_per_s": r["walk_steps_per_s"],
                "ms_per_step": r["ms_per_step"], "steps": r["steps"], "warmup": r["warmup"],
                "batch_walks": r["config"]["batch_walks"], "mean_loss": r["mean_loss"],
                "gpu_launches": r["gpu_launches"], "table_dtype": tdt, "n_nodes": r["config"]["n_nodes"],
                "n_edges": r["config"]["n_edges"], "roofline": r["roofline"], "walk": r["walk"],
                "clocks": r["clocks"], "leg_s": round(time.time() - t0, 1)}
        out["per_config"] = legs
    if out is not None:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    from paper_2407_15452_b200.workloads import WORKLOADS
    wl = WORKLOADS[args.workload]
    if args.dim is not None:
        import dataclasses
        wl = dataclasses.replace(wl, dim=args.dim)
    if args.stage == "row-updates" and args.impl != "reference":
        return run_row_update_probe(args)
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
