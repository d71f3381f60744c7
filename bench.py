#!/usr/bin/env python
"""Benchmark of the pivoted (PBP) fully-connected layer on B200.

A step is one forward call of one layer: y = act(W x + b), batch 1, on the
8192 x 8192 fp16 workload (tile 64, k of 128 tiles kept per block-row; k=128
is density 1.0).  Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--k 128] [--impl reference]

Device-timed `value` (us per layer): a CUDA graph of K forward calls that rotate
over enough independent copies of the layer that no call finds its weights in
L2 is replayed back to back; every replay is one timed region of exactly K
steps between two CUDA events on the launching stream, and `value` is the
median region's time per call (Section 5 of the paper averages 2,500 calls;
the regions together hold at least that many).  `roofline.isolated_us` is the
same layer as single launches without programmatic overlap, one event pair
per call.  `e2e` is the same call made from host buffers through the library's
host-buffer entry point (pinned host -> device copy, forward, device -> host
copy, synchronise).  With several GPUs every rank runs an independent replica
(no collective on the data path); the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import ctypes
import hashlib
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
MIN_TIMED_CALLS = 2500          # the paper's latency figures average 2,500 calls (Section 5)
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the headline kernel (ncu, profiles/
# stream_f16_cfg5_k128_batch1.md), valid for the kernel source with this SHA-256 prefix only
STREAM_TRAFFIC = {"bytes": 139.76e6, "source": "paper_1712_01084_b200/csrc/pp_stream.cu", "sha256_16": "b0612e7a227b1eb7"}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "tflops": float(d["bf16_tflops"]), "kind": "measured"}
    except Exception:
        return {"hbm_gbs": 6650.0, "tflops": 1590.0, "kind": "fallback"}


def traffic_if_current():
    """The recorded DRAM traffic, or None once the kernel source differs from the one the counters were taken on."""
    try:
        with open(os.path.join(ROOT, STREAM_TRAFFIC["source"]), "rb") as f:
            sha = hashlib.sha256(f.read()).hexdigest()[:16]
    except OSError:
        return None
    return STREAM_TRAFFIC["bytes"] if sha == STREAM_TRAFFIC["sha256_16"] else None


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


def n_tile_col(lay):
    """Length of the padded per-block-row tile-column index arrays (each block-row's list padded to 4 entries)."""
    counts = np.bincount(np.asarray(lay.tile_list)[:, 0], minlength=lay.Mb) if lay.T else np.zeros(lay.Mb, dtype=np.int64)
    return int(((counts + 3) // 4 * 4).sum())


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


# ----------------------------------------------------------------------------- device timing
def _pct(v, q):
    return float(np.percentile(np.asarray(v, dtype=np.float64), q))


GRAPH_CALLS = 1000        # calls captured in one CUDA graph; a longer region replays it several times


def region_plan(calls_per_region, graph_calls=GRAPH_CALLS):
    """A region of `calls_per_region` calls as (calls in the main graph, replays of it, calls in the remainder graph)."""
    main = min(calls_per_region, graph_calls)
    return main, calls_per_region // main, calls_per_region % main


def time_regions(torch, enqueue, calls_per_region, regions, warm_calls=0, before=None, after=None):
    """`enqueue(i, stream_ptr)` makes call i.  A region is exactly `calls_per_region` calls replayed from CUDA
    graphs (one graph when it has at most GRAPH_CALLS calls); `regions` regions run back to back, separated by
    events on the launching stream.  Returns the regions' times per call in us (a list), the device time from
    the first to the last event in ms, and the wall-clock interval of the timed part."""
    stream = torch.cuda.Stream()
    main, replays, rem = region_plan(calls_per_region)
    with torch.cuda.stream(stream):
        sp = ctypes.c_void_p(stream.cuda_stream)
        for i in range(max(warm_calls, 3)):
            enqueue(i, sp)                               # untimed warm-up, plain launches
        stream.synchronize()
        graphs = {}
        for n in {main, rem} - {0}:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                cp = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
                for i in range(n):
                    enqueue(i, cp)
            graphs[n] = g
        graphs[main].replay()                            # one untimed replay
        stream.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(regions + 1)]
        if before:
            before()
        torch.cuda.synchronize()
        w0 = time.time()
        ev[0].record(stream)
        for r in range(regions):
            for _ in range(replays):
                graphs[main].replay()
            if rem:
                graphs[rem].replay()
            ev[r + 1].record(stream)
        torch.cuda.synchronize()
        w1 = time.time()
        if after:
            after()
    per_call = [ev[r].elapsed_time(ev[r + 1]) * 1e3 / calls_per_region for r in range(regions)]
    return per_call, ev[0].elapsed_time(ev[regions]), (w0, w1)


def time_single_calls(torch, enqueue, n, warm=8):
    """Device time of single launches, one event pair per call (no overlap with a predecessor): us per call, a list."""
    stream = torch.cuda.Stream()
    out = []
    with torch.cuda.stream(stream):
        sp = ctypes.c_void_p(stream.cuda_stream)
        for i in range(warm):
            enqueue(i, sp)
        stream.synchronize()
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        for i, (a, b) in enumerate(pairs):
            a.record(stream)
            enqueue(i, sp)
            b.record(stream)
        stream.synchronize()
        out = [a.elapsed_time(b) * 1e3 for a, b in pairs]
    return out


def quick_us(torch, enqueue, calls_per_region, regions=12):
    """Median region time per call (us) of `time_regions` for the secondary tables."""
    per_call, _, _ = time_regions(torch, enqueue, calls_per_region, regions, warm_calls=min(calls_per_region, 8))
    return statistics.median(per_call)


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


def _check_status(pb, st, where="forward"):
    if st != 0:
        raise pb.PPError(st, where)


class LayerSet:
    """A layer and enough independent device copies of it that rotating calls never find their weights in L2."""

    def __init__(self, pb, lay):
        self.lay = lay
        first = pb.Layer.from_synth(lay)
        wbytes = max(1, lay.T * lay.B * lay.B * lay.tile_values.dtype.itemsize)
        self.weight_bytes = wbytes
        R = max(2, -(-2 * L2_BYTES // wbytes) + 1)
        self.layers = [first] + [first.clone() for _ in range(R - 1)]
        self.ntc = n_tile_col(lay)

    def __len__(self):
        return len(self.layers)

    def close(self):
        for l in self.layers:
            l.close()
        self.layers = []


def forward_enqueue(pb, ls, x, y, batch, fn=None, rotate=True):
    fn = fn or pb.lib().pp_forward
    hs = [l._h for l in ls.layers]
    R = len(hs)
    xp, yp, act = ctypes.c_void_p(x.data_ptr()), ctypes.c_void_p(y.data_ptr()), int(ls.lay.act)

    def enqueue(i, sp):
        _check_status(pb, fn(hs[i % R] if rotate else hs[0], xp, yp, batch, act, sp))
    return enqueue


def calls_for(R, want=64):
    """Calls per graph: a multiple of the number of copies, about `want`."""
    return R * max(1, want // R)


def roof_fields(peaks, abytes, us, flops=None):
    gbs = abytes / us / 1e3
    d = {"us": round(us, 3), "GBps": round(gbs, 1), "frac": round(gbs / peaks["hbm_gbs"], 3)}
    if flops is not None:
        d["tensor_frac"] = round(flops / (us * 1e-6) / 1e12 / peaks["tflops"], 3)
    return d


def paper_geometry(pb, torch, synth, sizes=(64, 128, 256, 512, 1024, 2048, 4096), per_sides=(32, 16, 8, 4)):
    """The geometry the paper itself measures (Section 5): size x size, 1/fill-in square blocks on the diagonal
    of the pivoted matrix, batch 1, here fp32.  Per case: this library's kernels (blocks through
    pp_layer_create_blocks, grid = block edge clamped to 16..64) and the plain kernels of the layout study: the
    three physical layouts of Section 4.1.1 ("brc", "bcr", "cbr") with a lane per output row ("rows") and with
    the lanes of a warp along the columns ("k").  "warm" repeats one layer as the paper's 2,500-call average does;
    "cold" rotates copies that together exceed twice the L2 (given where at most 96 copies do)."""
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
            warm = quick_us(torch, lambda i, sp: _check_status(pb, fn(L0._h, x.data_ptr(), y.data_ptr(), 1, 0, sp)), 64)
            row = {"block_edge": edge, "grid": grid, "block_bytes": lay.block_bytes, "us_warm": round(warm, 3)}
            R = -(-2 * L2_BYTES // max(1, lay.block_bytes)) + 1
            if R <= 96:
                reps = [L0] + [L0.clone() for _ in range(R - 1)]
                cold = quick_us(torch, lambda i, sp: _check_status(pb, fn(reps[i % R]._h, x.data_ptr(), y.data_ptr(), 1, 0, sp)), R)
                row.update({"us_cold": round(cold, 3), "GBps_cold": round(lay.block_bytes / cold / 1e3, 1), "copies": R})
                for r in reps[1:]:
                    r.close()
            L0.close()
            x1, y1 = x.reshape(-1), y.reshape(-1)
            fl = pb.lib().pp_layout_forward
            for mname, mapping in (("rows", pb.PP_MAP_ROWS_PER_LANE), ("k", pb.PP_MAP_LANES_ALONG_K)):
                for name, layout in (("brc", pb.PP_LAYOUT_BRC), ("bcr", pb.PP_LAYOUT_BCR), ("cbr", pb.PP_LAYOUT_CBR)):
                    K = pb.LayoutStudy(size, per_side, layout, mapping, lay.row_perm, lay.col_perm, lay.block_values)
                    row[f"{mname}_{name}_us_warm"] = round(quick_us(
                        torch, lambda i, sp: _check_status(pb, fl(K._h, x1.data_ptr(), y1.data_ptr(), sp)), 64), 3)
                    K.close()
            geo[f"size{size}_fill{100.0 / per_side:g}"] = row
    return geo


def density_sweep(pb, torch, synth, peaks, headline_k, headline_us):
    """Config 5 at every density and batch 1 / 16 / 128: us (cold), fraction of the measured copy bandwidth on
    algorithmic bytes, tensor fraction for the batched calls, speedup against density 1 at the same batch and
    linearity = speedup x density (1 = latency proportional to density)."""
    table = {}
    for k in (128, 64, 32, 16, 8):
        wl = synth.config5(k=k, batch=128)
        lay = wl.layers[0]
        ls = LayerSet(pb, lay)
        R = len(ls)
        row = {}
        for batch in (1, 16, 128):
            x = torch.from_numpy(np.ascontiguousarray(wl.x[:batch])).cuda()
            y = torch.empty((batch, lay.M), dtype=torch.float32, device="cuda")
            if batch == 1 and k == headline_k and headline_us is not None:
                us = headline_us
            else:
                us = quick_us(torch, forward_enqueue(pb, ls, x, y, batch), calls_for(R, 64 if batch == 1 else 16),
                              regions=12 if batch == 1 else 6)
            ab = algorithmic_bytes(lay, batch, ls.ntc)
            row[f"b{batch}"] = roof_fields(peaks, ab, us, None if batch == 1 else 2.0 * lay.T * lay.B * lay.B * batch)
        ls.close()
        table[f"{k / 128:.4g}"] = row
    for batch in (1, 16, 128):
        base = table["1"][f"b{batch}"]["us"]
        for key, row in table.items():
            sp = base / row[f"b{batch}"]["us"]
            row[f"b{batch}"]["speedup"] = round(sp, 3)
            row[f"b{batch}"]["linearity"] = round(sp * float(key), 3)
    return table


def permutation_overhead(pb, torch, synth):
    """Section 5's permutation-overhead experiment: the same layer with random and with identity index arrays."""
    out = {}
    for name, make in (("cfg5_k16_batch1", lambda **kw: synth.config5(k=16, batch=1, **kw)),
                       ("cfg1_batch1", lambda **kw: synth.config1(**kw))):
        row = {}
        for kind, kw in (("random", {}), ("identity", {"identity_perms": True})):
            wl = make(**kw)
            ls = LayerSet(pb, wl.layers[0])
            x = torch.from_numpy(wl.x).cuda()
            y = torch.empty((1, wl.layers[0].M), dtype=torch.float32, device="cuda")
            row[f"us_{kind}"] = round(quick_us(torch, forward_enqueue(pb, ls, x, y, 1), calls_for(len(ls))), 3)
            ls.close()
        row["overhead"] = round(row["us_random"] / row["us_identity"] - 1.0, 3)
        out[name] = row
    return out


def inputs_ready(pb, torch, synth, peaks):
    """The headline layer and sparser ones when the input does not come from the previous call (independent
    requests whose inputs sit in device memory beforehand; tuning key 17): x is fetched ahead of the dependency
    wait, only the writes wait.  Beside the headline, which keeps the dependent case."""
    out = {}
    for k in (128, 32, 16):
        wl = synth.config5(k=k, batch=1)
        lay = wl.layers[0]
        ls = LayerSet(pb, lay)
        x = torch.from_numpy(wl.x).cuda()
        y = torch.empty((1, lay.M), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        pb.pp_set_tuning(17, 1)
        try:
            us = quick_us(torch, forward_enqueue(pb, ls, x, y, 1), calls_for(len(ls), 240))
        finally:
            pb.pp_set_tuning(17, 0)
        out[f"cfg5_k{k}_batch1"] = roof_fields(peaks, algorithmic_bytes(lay, 1, ls.ntc), us)
        ls.close()
    return out


def other_workloads(pb, torch, synth, peaks):
    """Latency of the other synthetic workloads: cold (calls rotate over copies of the layers that together
    exceed twice the L2) and warm (one copy, weights may sit in L2), with the fraction of the measured copy
    bandwidth that the cold figure is on the workload's algorithmic bytes."""
    out = {}

    def layer_case(name, wl, batch, pivoted=False):
        lay = wl.layers[0]
        ls = LayerSet(pb, lay)
        x = torch.from_numpy(wl.x).cuda()
        y = torch.empty((batch, -(-lay.M // lay.B) * lay.B), dtype=torch.float32, device="cuda")
        fn = pb.lib().pp_forward_pivoted if pivoted else pb.lib().pp_forward
        cold = quick_us(torch, forward_enqueue(pb, ls, x, y, batch, fn), calls_for(len(ls), 64 if batch == 1 else 16))
        warm = quick_us(torch, forward_enqueue(pb, ls, x, y, batch, fn, rotate=False), 64 if batch == 1 else 16)
        ab = algorithmic_bytes(lay, batch, ls.ntc)
        row = roof_fields(peaks, ab, cold, None if batch == 1 else 2.0 * lay.T * lay.B * lay.B * batch)
        row["us_warm"] = round(warm, 3)
        row["kernel"] = ls.layers[0].launch_info(batch)["kernel"]
        out[name] = row
        ls.close()

    layer_case("cfg1_fc1024_f32_b32_d25_batch1", synth.config1(), 1)
    layer_case("cfg2_fc4096_f32_b64_d12.5_batch1", synth.config2(), 1)
    layer_case("cfg5_k128_batch128_pivoted_output", synth.config5(k=128, batch=128), 128, pivoted=True)

    for batch in (1, 8):
        wl = synth.config3(batch=batch)
        wbytes = sum(l.T * l.B * l.B * 2 for l in wl.layers)
        abytes = sum(algorithmic_bytes(l, batch, n_tile_col(l)) for l in wl.layers)
        R = -(-2 * L2_BYTES // wbytes) + 1
        chains = []
        for _ in range(R):
            layers = [pb.Layer.from_synth(l) for l in wl.layers] if not chains else [l.clone() for l in chains[0].layers]
            chains.append(pb.Chain(layers, [l.act for l in wl.layers], max_batch=8))
        x = torch.from_numpy(wl.x).cuda()
        y = torch.empty((batch, wl.layers[-1].M), dtype=torch.float32, device="cuda")
        fn = pb.lib().pp_chain_forward
        cold = quick_us(torch, lambda i, sp: _check_status(pb, fn(chains[i % R]._h, x.data_ptr(), y.data_ptr(), batch, sp)), R * 2)
        warm = quick_us(torch, lambda i, sp: _check_status(pb, fn(chains[0]._h, x.data_ptr(), y.data_ptr(), batch, sp)), 32)
        row = roof_fields(peaks, abytes, cold)
        row.update({"us_warm": round(warm, 3), "layers": 3})
        out[f"cfg3_chain_batch{batch}"] = row
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
    us = quick_us(torch, lambda i, sp: _check_status(pb, fn(cell._h, xs.data_ptr(), h.data_ptr(), c.data_ptr(), 256, sp)), 1, regions=5)
    wb = lay.T * lay.B * lay.B * 2
    out["cfg4_lstm_256_steps"] = {"us_per_step": round(us / 256, 3), "us_total": round(us, 1),
                                  "frac_if_weights_came_from_hbm": round(wb / (us / 256) / 1e3 / peaks["hbm_gbs"], 3),
                                  "note": "weights resident on chip; the fraction is a reference line, not a bound"}
    cell.close(); L.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--k", type=int, default=128, help="kept tiles per block-row (of 128)")
    ap.add_argument("--no-sweep", action="store_true", help="skip the density sweep")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline")
    ap.add_argument("--no-configs", action="store_true", help="skip the other synthetic workloads")
    ap.add_argument("--geometry", default=None, metavar="SIZE:BLOCKS|all",
                    help="only time the paper's square-block geometry (one case such as 2048:4, or all) and print that table")
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
        pb.lib()
        if args.geometry == "all":
            geo = paper_geometry(pb, torch, synth)
        else:
            size, per_side = (int(v) for v in args.geometry.split(":"))
            geo = paper_geometry(pb, torch, synth, (size,), (per_side,))
        print(json.dumps({"paper_geometry_f32_batch1": geo}))
        return
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    pb.lib()
    peaks = measured_peaks()

    def barrier():
        if world > 1:
            dist.barrier()

    # ---- headline: K calls per timed region, regions repeated until they hold at least MIN_TIMED_CALLS calls
    wl = synth.config5(k=args.k, batch=1)
    lay = wl.layers[0]
    ls = LayerSet(pb, lay)
    x = torch.from_numpy(wl.x).cuda()
    y = torch.empty((1, lay.M), dtype=torch.float32, device="cuda")
    regions = max(5, -(-MIN_TIMED_CALLS // args.steps))
    sampler = ClockSampler(local_rank)
    time.sleep(0.3)
    per_call, total_ms, (w0, w1) = time_regions(torch, forward_enqueue(pb, ls, x, y, 1), args.steps, regions,
                                                warm_calls=args.warmup, before=barrier, after=barrier)
    clocks = sampler.stop(w0, w1)
    us_step = max_over_ranks(statistics.median(per_call), world)     # one step = one layer on every rank
    value = job_value(us_step, world)
    info = ls.layers[0].launch_info(1)

    # ---- the same layer as single launches with no programmatic overlap: one cold call at a time
    pb.pp_set_tuning(8, 0)
    try:
        iso = time_single_calls(torch, forward_enqueue(pb, ls, x, y, 1), 200)
    finally:
        pb.pp_set_tuning(8, 1)
    iso_us = statistics.median(iso)

    # ---- end to end from host buffers through the library's host-buffer call
    n_e2e = min(max(args.steps, 50), 300)
    xh = torch.from_numpy(wl.x).pin_memory()
    yh = torch.empty((1, lay.M), dtype=torch.float32).pin_memory()
    t0 = time.perf_counter()
    for i in range(5 + n_e2e):
        if i == 5:
            torch.cuda.synchronize()
            t0 = time.perf_counter()
        pb.pp_forward_host(ls.layers[i % len(ls)], xh, lay.act, out=yh)
    e2e_us = max_over_ranks((time.perf_counter() - t0) / n_e2e * 1e6, world)

    abytes = algorithmic_bytes(lay, 1, ls.ntc)
    achieved = abytes / (us_step * 1e-6) / 1e9
    out = {
        "metric": METRIC, "value": value, "unit": "us", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": us_step / 1e3, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f16 weights, f32 accumulate", "data": "synthetic",
        "config": {"workload": wl.name, "batch": 1, "M": lay.M, "N": lay.N, "B": lay.B,
                   "tiles_per_block_row": args.k, "density": args.k / 128, "launch": "cuda_graph",
                   "l2": f"inputs larger than L2: calls rotate over {len(ls)} independent copies of the "
                         f"layer ({len(ls) * ls.weight_bytes / 2**20:.0f} MiB of weights)",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "gpu_launches": args.steps,
        "timing": {"regions": regions, "calls_per_region": args.steps, "calls_total": regions * args.steps,
                   "value_is": "median region, us per call", "us_p10": round(_pct(per_call, 10), 3),
                   "us_p50": round(_pct(per_call, 50), 3), "us_p90": round(_pct(per_call, 90), 3),
                   "us_mean": round(total_ms * 1e3 / (regions * args.steps), 3)},
        "e2e": {"value": e2e_us / world, "unit": "us", "h2d_bytes_per_step": int(wl.x.nbytes),
                "d2h_bytes_per_step": int(lay.M * 4), "steps": n_e2e},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": achieved / peaks["hbm_gbs"], "peak_kind": f"of {peaks['kind']}",
                     "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS, "algorithmic_bytes_per_launch": abytes,
                     "kernel": f"stream_f16_kernel<{info['ring_depth']}>, {info['ctas']} CTAs, "
                               f"{info['smem_bytes']} B shared memory, programmatic overlap with the previous call",
                     "isolated_us": round(iso_us, 3), "isolated_frac": abytes / iso_us / 1e3 / peaks["hbm_gbs"],
                     "isolated_is": "median of 200 single cold launches without programmatic overlap, one event pair each",
                     "traffic": traffic_if_current() if args.k == 128 else None},
        "clocks": clocks,
    }
    ls.close()
    solo = rank == 0 and world == 1
    if solo and not args.no_cpu:
        out["cpu_baseline"] = cpu_baseline(lay, wl.x)
    if solo and not args.no_configs:
        out["permutation_overhead"] = permutation_overhead(pb, torch, synth)
        out["inputs_ready_before_the_stream"] = inputs_ready(pb, torch, synth, peaks)
        out["other_workloads"] = other_workloads(pb, torch, synth, peaks)
    if solo and not args.no_sweep:
        out["density_sweep"] = density_sweep(pb, torch, synth, peaks, args.k, us_step)

    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
