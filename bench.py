#!/usr/bin/env python
"""Benchmark of the pivoted (PBP) fully-connected layer on B200.

A step is one forward call of one layer: y = act(W x + b), batch 1, on the
8192 x 8192 fp16 workload (tile 64, k of 128 tiles kept per block-row; k=128
is density 1.0).  Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--k 128] [--impl reference]

Device-timed `value` (us per layer) replays a CUDA graph of forward calls that
rotate over enough independent copies of the layer that no call finds its
weights in L2.  `e2e` is the same call made from host buffers through the
Python binding (pinned host -> device copy, forward, device -> host read, sync).
With several GPUs every rank runs an independent replica (no collective on the
data path); the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import ctypes
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

METRIC = "pivoted_fc_us_per_layer_batch1"
L2_BYTES = 126 * 1024 * 1024
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the headline kernel (ncu; see profiles/);
# None while the kernel has changed since the counters were taken
STREAM_TRAFFIC_BYTES = 139.52e6


def measured_peak_gbs():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def algorithmic_bytes(lay, batch, n_tile_col):
    """Bytes one forward call must move: kept tiles, index arrays, x, y, permutations, bias."""
    esz = lay.tile_values.dtype.itemsize
    Mb, Nb = lay.Mb, lay.Nb
    b = lay.T * lay.B * lay.B * esz
    b += 4 * (n_tile_col + Mb + 1)
    b += lay.N * batch * esz + lay.M * batch * 4
    b += 4 * (Nb * lay.B + Mb * lay.B)
    b += 4 * lay.M if lay.bias is not None else 0
    return b


class ClockSampler:
    """nvidia-smi polling in a child process; killed by PID when done."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        rows = []
        for line in out.splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                ts = time.mktime(time.strptime(parts[0].split(".")[0], "%Y/%m/%d %H:%M:%S")) + \
                    float("0." + parts[0].split(".")[1])
                rows.append((ts, float(parts[1]), float(parts[2]), parts[4:8]))
            except Exception:
                continue
        inside = [r for r in rows if t0 <= r[0] <= t1]
        use = inside if len(inside) >= 3 else rows
        if not use:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for r in use for n, v in zip(names, r[3]) if v.lower().startswith("active")})
        return {"sm_mhz": statistics.median(r[1] for r in use), "sm_max_mhz": use[0][2], "reasons": reasons,
                "samples": len(use), "window": "timed region" if use is inside else "whole run"}


def cpu_baseline(lay, x, budget_s=12.0):
    """The oracle as it stands, on this host: dense fp64 reconstruction, then matrix-vector products."""
    from oracle import pp_oracle as po
    cores = os.cpu_count() or 1
    t0 = time.perf_counter()
    W = po.reconstruct(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, lay.tile_list, lay.tile_values)
    t_rec = time.perf_counter() - t0
    x64 = x.astype(np.float64)
    po.dense_forward(W, lay.bias, x64, lay.act, threads=cores)
    reps, t_acc = 0, 0.0
    while t_acc < budget_s and reps < 30:
        t0 = time.perf_counter()
        po.dense_forward(W, lay.bias, x64, lay.act, threads=cores)
        t_acc += time.perf_counter() - t0
        reps += 1
    return {"value": t_acc / reps * 1e6, "unit": "us", "cores": cores, "kind": "oracle",
            "sample": f"{reps} full dense fp64 matrix-vector products of the same layer "
                      f"(dense reconstruction, {t_rec:.2f} s, done once and not counted)"}


def run_reference(args, rank):
    """Reference arm: the CPU oracle timed on the host cores, same workload, metric and unit."""
    if rank != 0:
        return
    from oracle import pp_oracle as po
    from paper_1712_01084_b200 import synth
    wl = synth.config5(k=args.k, batch=1)
    lay = wl.layers[0]
    cores = os.cpu_count() or 1
    W = po.reconstruct(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, lay.tile_list, lay.tile_values)
    x64 = wl.x.astype(np.float64)
    po.dense_forward(W, None, x64, lay.act, threads=cores)
    t0 = time.perf_counter()
    po.dense_forward(W, None, x64, lay.act, threads=cores)
    t_full = time.perf_counter() - t0
    # each step is the whole layer on all cores when that fits the budget of one step, else a sample of output
    # rows (one thread) sized from a timed probe, so that the whole run stays near two minutes
    budget = 120.0 / max(1, args.steps + args.warmup)
    rows_all = np.random.default_rng(0).permutation(lay.M).astype(np.int32)
    if t_full <= budget:
        n_rows = lay.M
    else:
        probe = rows_all[:64]
        po.dense_forward_rows(W, None, x64, lay.act, probe)
        t0 = time.perf_counter()
        po.dense_forward_rows(W, None, x64, lay.act, probe)
        t_row = (time.perf_counter() - t0) / probe.size
        n_rows = int(min(lay.M, max(1, budget / max(t_row, 1e-9))))
    rows = rows_all[:n_rows].copy()
    run = (lambda: po.dense_forward(W, None, x64, lay.act, threads=cores)) if n_rows >= lay.M else \
          (lambda: po.dense_forward_rows(W, None, x64, lay.act, rows))
    used = cores if n_rows >= lay.M else 1
    for _ in range(args.warmup):
        run()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run()
    t = (time.perf_counter() - t0) / args.steps
    us = t * 1e6 * (lay.M / min(n_rows, lay.M))
    sample = f"{min(n_rows, lay.M)} of {lay.M} output rows per step, scaled to the full layer"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": us, "unit": "us", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "batch": 1, "M": lay.M, "N": lay.N, "B": lay.B, "tiles_per_block_row": args.k},
        "cpu_baseline": {"value": us, "unit": "us", "cores": used, "kind": "oracle", "sample": sample},
        "e2e": {"value": us, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def time_graph(pb, torch, replicas, x, y, act, steps, warmup, chunk=500):
    """Device time of `steps` forward calls (rotating replicas) replayed from CUDA graphs."""
    fn = pb.lib().pp_forward
    xp, yp = ctypes.c_void_p(x.data_ptr()), ctypes.c_void_p(y.data_ptr())
    handles = [r._h for r in replicas]
    R = len(handles)

    def enqueue(n, start, stream_ptr):
        for s in range(n):
            st = fn(handles[(start + s) % R], xp, yp, 1, act, stream_ptr)
            if st != 0:
                raise pb.PPError(st, "pp_forward")

    stream = torch.cuda.Stream()
    graphs = {}
    with torch.cuda.stream(stream):
        sp = ctypes.c_void_p(stream.cuda_stream)
        enqueue(max(warmup, 3), 0, sp)              # untimed warm-up, plain launches
        stream.synchronize()
        chunk = min(chunk, steps)
        chunk -= chunk % R if chunk > R else 0
        chunk = max(chunk, 1)
        for n in {chunk, steps % chunk} - {0}:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                enqueue(n, 0, ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
            graphs[n] = g
        graphs[chunk].replay()                      # one untimed replay
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        return stream, graphs, chunk, e0, e1


def max_over_ranks(value, world, device="cuda"):
    """The slowest rank's figure (every rank runs an independent replica; the job is as slow as that one)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(us_step_max, world):
    """Whole-job microseconds per layer: `world` replicas finish one layer each per (slowest) step."""
    return us_step_max / world


def time_enqueue(torch, enqueue, calls_per_graph, replays=20):
    """Mean device time (us) of one call: `enqueue(i, stream_ptr)` is captured `calls_per_graph`
    times into a CUDA graph that is replayed `replays` times between two events."""
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        sp = ctypes.c_void_p(stream.cuda_stream)
        for i in range(calls_per_graph):
            enqueue(i, sp)                               # warm-up, plain launches
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            cp = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
            for i in range(calls_per_graph):
                enqueue(i, cp)
        g.replay()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(replays):
            g.replay()
        e1.record(stream)
        stream.synchronize()
    return e0.elapsed_time(e1) * 1e3 / (replays * calls_per_graph)


def paper_geometry(pb, torch, synth, sizes=(64, 128, 256, 512, 1024, 2048, 4096), per_sides=(32, 16, 8, 4)):
    """The geometry the paper itself measures (Section 5): size x size, 1/fill-in square blocks on the diagonal
    of the pivoted matrix, batch 1, here fp32.  Per case: this library's kernels (blocks through
    pp_layer_create_blocks, grid = block edge clamped to 16..64) and the paper's own kernel model (one thread
    group per block, one thread per output row) in its three physical layouts.  "warm" repeats one layer as the
    paper's 2,500-call average does; "cold" rotates copies that together exceed twice the L2 (given where at
    most 96 copies do)."""
    def check(st):
        if st != 0:
            raise pb.PPError(st, "forward")

    geo = {}
    for size in sizes:
        for per_side in per_sides:
            edge = size // per_side
            grid = 16 if edge <= 16 else 32 if edge <= 32 else 64
            wl = synth.paper_square(size, per_side, grid, wdtype="f32")
            lay = wl.layers[0]
            L0 = pb.Layer.from_synth(lay)
            x = torch.from_numpy(wl.x).cuda()
            y = torch.empty((1, size), dtype=torch.float32, device="cuda")
            fn = pb.lib().pp_forward
            warm = time_enqueue(torch, lambda i, sp: check(fn(L0._h, x.data_ptr(), y.data_ptr(), 1, 0, sp)), 64)
            row = {"block_edge": edge, "grid": grid, "block_bytes": lay.block_bytes, "us_warm": round(warm, 3)}
            R = -(-2 * L2_BYTES // max(1, lay.block_bytes)) + 1
            if R <= 96:
                reps = [L0] + [L0.clone() for _ in range(R - 1)]
                cold = time_enqueue(torch, lambda i, sp: check(fn(reps[i % R]._h, x.data_ptr(), y.data_ptr(), 1, 0, sp)), R)
                row.update({"us_cold": round(cold, 3), "GBps_cold": round(lay.block_bytes / cold / 1e3, 1), "copies": R})
                for r in reps[1:]:
                    r.close()
            L0.close()
            # the paper's own kernel (one thread group per block, one thread per output row) in its three layouts
            if edge <= 1024:
                x1, y1 = x.reshape(-1), y.reshape(-1)
                fl = pb.lib().pp_listing1_forward
                for name, layout in (("brc", pb.PP_LAYOUT_BRC), ("bcr", pb.PP_LAYOUT_BCR), ("cbr", pb.PP_LAYOUT_CBR)):
                    K = pb.Listing1(size, per_side, layout, lay.row_perm, lay.col_perm, lay.block_values)
                    row[f"listing1_{name}_us_warm"] = round(time_enqueue(
                        torch, lambda i, sp: check(fl(K._h, x1.data_ptr(), y1.data_ptr(), sp)), 64), 3)
                    K.close()
            geo[f"size{size}_fill{100.0 / per_side:g}"] = row
    return geo


def other_workloads(pb, torch, synth):
    """Latency of the other synthetic workloads: cold (calls rotate over copies of the layers that
    together exceed twice the L2) and warm (one copy, weights may sit in L2)."""
    out = {}

    def check(st):
        if st != 0:
            raise pb.PPError(st, "forward")

    def layer_case(name, wl, batch, pivoted=False):
        lay = wl.layers[0]
        L0 = pb.Layer.from_synth(lay)
        wbytes = lay.T * lay.B * lay.B * lay.tile_values.dtype.itemsize
        R = max(2, -(-2 * L2_BYTES // wbytes) + 1)
        reps = [L0] + [L0.clone() for _ in range(R - 1)]
        x = torch.from_numpy(wl.x).cuda()
        y = torch.empty((batch, -(-lay.M // lay.B) * lay.B), dtype=torch.float32, device="cuda")
        fn = pb.lib().pp_forward_pivoted if pivoted else pb.lib().pp_forward
        cold = time_enqueue(torch, lambda i, sp: check(fn(reps[i % R]._h, x.data_ptr(), y.data_ptr(), batch, lay.act, sp)), R * max(1, 64 // R))
        warm = time_enqueue(torch, lambda i, sp: check(fn(L0._h, x.data_ptr(), y.data_ptr(), batch, lay.act, sp)), 64)
        pk = pb.Packed(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, lay.tile_list, lay.tile_values, lay.bias)
        ab = algorithmic_bytes(lay, batch, pk.n_tile_col)
        out[name] = {"us_cold": round(cold, 3), "us_warm": round(warm, 3), "GBps_cold": round(ab / cold / 1e3, 1),
                     "algorithmic_bytes": ab, "copies": R}
        for r in reps:
            r.close()

    layer_case("cfg1_fc1024_f32_b32_d25_batch1", synth.config1(), 1)
    layer_case("cfg2_fc4096_f32_b64_d12.5_batch1", synth.config2(), 1)
    for batch in (16, 128):
        layer_case(f"cfg5_fc8192_f16_b64_k128_batch{batch}", synth.config5(k=128, batch=batch), batch)
    # the same product with the output left in pivoted row order (output permutation elimination)
    layer_case("cfg5_fc8192_f16_b64_k128_batch128_pivoted_output", synth.config5(k=128, batch=128), 128, pivoted=True)
    layer_case("cfg5_fc8192_f16_b64_k32_batch128", synth.config5(k=32, batch=128), 128)

    out["paper_geometry_f32_batch1"] = paper_geometry(pb, torch, synth)

    for batch in (1, 8):
        wl = synth.config3(batch=batch)
        wbytes = sum(l.T * l.B * l.B * 2 for l in wl.layers)
        R = -(-2 * L2_BYTES // wbytes) + 1
        chains = []
        for _ in range(R):
            layers = [pb.Layer.from_synth(l) for l in wl.layers] if not chains else [l.clone() for l in chains[0].layers]
            chains.append(pb.Chain(layers, [l.act for l in wl.layers], max_batch=8))
        x = torch.from_numpy(wl.x).cuda()
        y = torch.empty((batch, wl.layers[-1].M), dtype=torch.float32, device="cuda")
        fn = pb.lib().pp_chain_forward
        cold = time_enqueue(torch, lambda i, sp: check(fn(chains[i % R]._h, x.data_ptr(), y.data_ptr(), batch, sp)), R * 2)
        warm = time_enqueue(torch, lambda i, sp: check(fn(chains[0]._h, x.data_ptr(), y.data_ptr(), batch, sp)), 32)
        out[f"cfg3_chain_batch{batch}"] = {"us_cold": round(cold, 3), "us_warm": round(warm, 3), "layers": 3,
                                            "us_per_layer_cold": round(cold / 3, 3), "tile_bytes": wbytes, "copies": R}
        for c in chains:
            c.close()
            for l in c.layers:
                l.close()

    wl = synth.config4(steps=256)
    lay, H, I = wl.layers[0], wl.extra["H"], wl.extra["I"]
    L = pb.Layer.from_synth(lay)
    cell = pb.Lstm(L, I, H, max_steps=256)
    xs = torch.from_numpy(wl.x).cuda()
    h = torch.zeros(H, dtype=torch.float16, device="cuda")
    c = torch.zeros(H, dtype=torch.float32, device="cuda")
    fn = pb.lib().pp_lstm_forward
    us = time_enqueue(torch, lambda i, sp: check(fn(cell._h, xs.data_ptr(), h.data_ptr(), c.data_ptr(), 256, sp)), 1, replays=5)
    out["cfg4_lstm_256_steps"] = {"us_total": round(us, 1), "us_per_step": round(us / 256, 3),
                                  "tile_bytes_per_step": lay.T * lay.B * lay.B * 2, "note": "one cooperative kernel for all steps, gate weights resident in shared memory"}
    cell.close(); L.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=200)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--k", type=int, default=128, help="kept tiles per block-row (of 128)")
    ap.add_argument("--no-sweep", action="store_true", help="skip the density sweep")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline")
    ap.add_argument("--no-configs", action="store_true", help="skip the other synthetic workloads")
    ap.add_argument("--geometry", default=None, metavar="SIZE:BLOCKS",
                    help="only time the paper's square-block geometry for one case (e.g. 2048:4) and print that table")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_1712_01084_b200 import binding as pb
    from paper_1712_01084_b200 import synth

    torch.cuda.set_device(local_rank)
    if args.geometry:
        size, per_side = (int(v) for v in args.geometry.split(":"))
        pb.lib()
        print(json.dumps({"paper_geometry_f32_batch1": paper_geometry(pb, torch, synth, (size,), (per_side,))}))
        return
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    pb.lib()

    def barrier():
        if world > 1:
            dist.barrier()

    def build(k):
        wl = synth.config5(k=k, batch=1)
        lay = wl.layers[0]
        L0 = pb.Layer.from_synth(lay)
        pk_bytes = lay.T * lay.B * lay.B * 2
        R = max(2, -(-2 * L2_BYTES // pk_bytes) + 1)
        reps = [L0] + [L0.clone() for _ in range(R - 1)]
        return wl, lay, reps

    def time_config(k, steps, warmup, sample_clocks=False):
        wl, lay, reps = build(k)
        x = torch.from_numpy(wl.x).cuda()
        y = torch.empty((1, lay.M), dtype=torch.float32, device="cuda")
        stream, graphs, chunk, e0, e1 = time_graph(pb, torch, reps, x, y, lay.act, steps, warmup)
        sampler = ClockSampler(local_rank) if sample_clocks else None
        if sampler:
            time.sleep(0.3)
        barrier()
        torch.cuda.synchronize()
        w0 = time.time()
        with torch.cuda.stream(stream):
            e0.record(stream)
            for _ in range(steps // chunk):
                graphs[chunk].replay()
            if steps % chunk:
                graphs[steps % chunk].replay()
            e1.record(stream)
        torch.cuda.synchronize()
        w1 = time.time()
        barrier()
        ms = e0.elapsed_time(e1)
        clocks = sampler.stop(w0, w1) if sampler else None
        return wl, lay, reps, x, y, ms, clocks

    wl, lay, reps, x, y, ms, clocks = time_config(args.k, args.steps, args.warmup, sample_clocks=True)
    ms = max_over_ranks(ms, world)
    us_step = ms * 1e3 / args.steps                      # one step = one layer on every rank
    value = job_value(us_step, world)

    # end to end from host buffers through the library's host-buffer call (pinned host -> device copy, forward,
    # device -> host copy, stream synchronize, all inside pp_forward_host)
    n_e2e = min(args.steps, 300)
    xh = torch.from_numpy(wl.x).pin_memory()
    yh = torch.empty((1, lay.M), dtype=torch.float32).pin_memory()
    for i in range(5 + n_e2e):
        if i == 5:
            torch.cuda.synchronize()
            t0 = time.perf_counter()
        pb.pp_forward_host(reps[i % len(reps)], xh, lay.act, out=yh)
    e2e_us = (time.perf_counter() - t0) / n_e2e * 1e6
    e2e_us = max_over_ranks(e2e_us, world)

    pk = pb.Packed(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, lay.tile_list, lay.tile_values, lay.bias)
    abytes = algorithmic_bytes(lay, 1, pk.n_tile_col)
    peak, peak_kind = measured_peak_gbs()
    achieved = abytes / (us_step * 1e-6) / 1e9
    out = {
        "metric": METRIC, "value": value, "unit": "us", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": us_step / 1e3, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f16 weights, f32 accumulate", "data": "synthetic",
        "config": {"workload": wl.name, "batch": 1, "M": lay.M, "N": lay.N, "B": lay.B,
                   "tiles_per_block_row": args.k, "density": args.k / 128, "launch": "cuda_graph",
                   "l2": f"inputs larger than L2: calls rotate over {len(reps)} independent copies of the "
                         f"layer ({len(reps) * lay.T * lay.B * lay.B * 2 / 2**20:.0f} MiB of weights)",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "gpu_launches": args.steps,
        "e2e": {"value": e2e_us / world, "unit": "us", "h2d_bytes_per_step": int(wl.x.nbytes),
                "d2h_bytes_per_step": int(lay.M * 4), "steps": n_e2e},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": f"of {peak_kind}", "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                     "algorithmic_bytes_per_launch": abytes, "kernel": "stream_f16_kernel<4>",
                     # dram__bytes_read.sum + dram__bytes_write.sum of one launch (ncu, profiles/stream_f16_cfg5_k128_batch1.md)
                     "traffic": STREAM_TRAFFIC_BYTES if args.k == 128 else None},
        "clocks": clocks,
    }

    if rank == 0 and not args.no_sweep and world == 1:
        sweep = {}
        base = None
        for k in (128, 64, 32, 16, 8):
            if k == args.k:
                us_k = us_step
                lay_k, n_tc = lay, pk.n_tile_col
            else:
                for r in reps:
                    r.close()
                wl_k, lay_k, reps, _, _, ms_k, _ = time_config(k, min(args.steps, 5000), min(args.warmup, 50))
                us_k = ms_k * 1e3 / min(args.steps, 5000)
                pkk = pb.Packed(lay_k.M, lay_k.N, lay_k.B, lay_k.row_perm, lay_k.col_perm, lay_k.tile_list,
                                lay_k.tile_values, None)
                n_tc = pkk.n_tile_col
            gbs = algorithmic_bytes(lay_k, 1, n_tc) / (us_k * 1e-6) / 1e9
            if k == 128:
                base = us_k
            sweep[f"{k / 128:.4g}"] = {"us": round(us_k, 3), "GBps": round(gbs, 1),
                                       "speedup_vs_dense": None if base is None else round(base / us_k, 3),
                                       "linearity": None if base is None else round(base / us_k * k / 128, 3)}
        out["density_sweep"] = sweep

    if rank == 0 and world == 1 and not args.no_configs:
        for r in reps:
            r.close()
        out["other_workloads"] = other_workloads(pb, torch, synth)

    if rank == 0 and world == 1 and not args.no_cpu:
        wl0 = synth.config5(k=args.k, batch=1)
        out["cpu_baseline"] = cpu_baseline(wl0.layers[0], wl0.x)

    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
