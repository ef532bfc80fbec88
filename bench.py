#!/usr/bin/env python
"""Benchmark of the batch-1 lattice GEMV path (one JSON line on stdout, rank 0).

A step is one pass over the workload's per-token sequence of lattice GEMVs (for the default
workload, the seven projections of a 4B-like decoder layer, issued as four row-concatenated
launches).  Inputs are synthetic and seeded; every row of the timed path is checked against the f64
CPU oracle before anything is timed (that check is also the cpu_baseline leg: the oracle's time on the
host cores); the comparison arms are then checked against the timed path's outputs.  Weights rotate through enough distinct copies that no
launch finds its records in L2.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

With --impl reference the CPU oracle itself is timed on the host cores (a bounded sample a step).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_02652_b200 import datagen  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
# DRAM bytes (read + write) per algorithmic byte of gemv_planes_kernel, from one ncu capture of the
# 8192 x 8192 launch (profiles/gemv_planes_kernel_config4_8192x8192.txt: 39.365 MB against 39.289 MB);
# traffic grows in proportion to the records streamed, so a launch's traffic is its bytes times this.
NCU_TRAFFIC_PER_ALGORITHMIC_BYTE = 39.3580 / 39.2888
# from the same capture: 5 847 216 warp instructions for 87 552 block columns (32 rows x 24 weights each), and the share
# of issue slots busy over the launch
NCU_WARP_INSTR_PER_CELL = 5826348 / 87552
NCU_ISSUE_BUSY_PCT = 56.6
METRIC = "us_per_lattice_gemv"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json, STREAM-style copy)"
    return 6650.0, "fallback (earlier measurement on this pool)"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while a region runs."""

    def __init__(self, index: int, period: float = 0.001):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.stop_flag, self.max_mhz = [], set(), threading.Event(), None
        self.period, self.index, self.ok = period, index, False
        try:
            import pynvml

            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    NAMES = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x10: "sync_boost",
             0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def run(self):
        if not self.ok:
            return
        while not self.stop_flag.is_set():
            try:
                self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
                r = self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                for bit, name in self.NAMES.items():
                    if r & bit and name != "gpu_idle":
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def result(self):
        self.stop_flag.set()
        if self.is_alive():
            self.join(timeout=2)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def gemv_bytes(rows: int, nb: int, bytes_per_block: int = 14) -> int:
    """Algorithmic bytes of one GEMV: records + fp16 scales + fp16 x + f32 y."""
    return bytes_per_block * rows * nb + 2 * rows + 2 * 24 * nb + 4 * rows


class Copy:
    """One resident copy of the workload: layouts, scales, x per launch group, outputs."""

    def __init__(self):
        self.launches = []      # per launch: dict(problems=ctypes array, x, k_padded, mats=[...], ys=[...], bufs=[...])


def build_inputs(wl, device):
    """Host-side codes/scales/x for every matrix; x is shared inside a launch group."""
    mats = []
    group_x = {}
    for m in wl.matrices:
        key = m.group if m.group >= 0 else ("solo", m.tensor_id)
        if key not in group_x:
            group_x[key] = datagen.make_x(m.k, m.k_padded, wl.seed, m.tensor_id)
        mats.append(dict(m=m, key=key, codes=datagen.make_codes(m.rows, m.nb, wl.seed, m.tensor_id, device=device),
                         scale=datagen.make_row_scale(m.rows, wl.seed, m.tensor_id), x=group_x[key]))
    return mats


def make_copies(B, ctx, mats, layout, ncopies, device, grouped=True):
    first = {}
    for e in mats:
        m = e["m"]
        first[m.tensor_id] = B.expand(ctx, layout, e["codes"], m.rows, m.nb)
    torch.cuda.synchronize()
    copies = []
    for c in range(ncopies):
        cp = Copy()
        keys = []
        for e in mats:
            k = e["key"] if grouped else ("solo", e["m"].tensor_id)
            if k not in keys:
                keys.append(k)
        for k in keys:
            members = [e for e in mats if (e["key"] if grouped else ("solo", e["m"].tensor_id)) == k]
            # x is the previous operator's output in a decoder: small and cache-resident.  One buffer a
            # launch, shared by every copy of the records; only the records (and scales) rotate.
            if ("x", k) not in first:
                first[("x", k)] = members[0]["x"].to(device)
            x = first[("x", k)]
            bufs = [first[e["m"].tensor_id] if c == 0 else first[e["m"].tensor_id].clone() for e in members]
            scales = [e["scale"].to(device) for e in members]
            ys = [torch.zeros(e["m"].rows, dtype=torch.float32, device=device) for e in members]
            probs = B.make_problems([(b, s, datagen.GAIN, y, e["m"].rows) for b, s, y, e in zip(bufs, scales, ys, members)])
            cp.launches.append(dict(problems=probs, x=x, k_padded=members[0]["m"].k_padded, mats=[e["m"] for e in members], ys=ys,
                                    bufs=bufs, scales=scales, members=members))
        copies.append(cp)
    return copies


def run_step(B, ctx, layout, cp):
    for ln in cp.launches:
        B.gemv_grouped(ctx, layout, ln["problems"], ln["x"], ln["k_padded"])


def verify(oracle, copies, threads, max_launches=None):
    """Every row of copy 0 (of its first max_launches launches) against the f64 oracle.
    Returns (worst normalised error, oracle seconds, blocks, GEMVs checked)."""
    worst, secs, blocks, gemvs = 0.0, 0.0, 0, 0
    for ln in copies[0].launches[:max_launches]:
        xh = ln["x"].cpu().numpy()
        for e, y in zip(ln["members"], ln["ys"]):
            m = e["m"]
            codes = e["codes"].cpu().numpy().astype(np.uint64)
            t0 = time.perf_counter()
            y_ref, wn, ab = oracle.matvec(codes, m.rows, m.nb, e["scale"].numpy(), datagen.GAIN, xh, nthreads=threads)
            secs += time.perf_counter() - t0
            blocks += m.blocks
            yv = y.cpu().numpy().astype(np.float64)
            denom = wn * float(np.linalg.norm(xh.astype(np.float64)))
            err = np.abs(yv - y_ref)
            ratio = np.where(denom > 0, err / np.where(denom > 0, denom, 1.0), 0.0)
            if not (np.isfinite(yv).all() and ratio.max() <= 1e-4 and (yv[denom == 0] == 0).all()):
                raise SystemExit(f"parity failure on {m.name}: normalised error {ratio.max():.3e}")
            worst = max(worst, float(ratio.max()))
            gemvs += 1
    return worst, secs, blocks, gemvs


def same_outputs(ref_copies, arm_copies, exact: bool) -> None:
    """An arm's outputs against those of the main arm, which the oracle checked row by row: bit for bit where the
    arithmetic is the same, else to 1e-4 of the output's scale (the GPU tests hold every arm to the oracle itself)."""
    for lr, la in zip(ref_copies[0].launches, arm_copies[0].launches):
        for m, yr, ya in zip(lr["mats"], lr["ys"], la["ys"]):
            if exact:
                ok = torch.equal(yr, ya)
            else:
                ok = bool(torch.isfinite(ya).all()) and float((yr - ya).abs().max()) <= 1e-4 * float(yr.abs().max()) + 1e-30
            if not ok:
                raise SystemExit(f"arm output differs from the checked one on {m.name}")


def capture_graphs(B, ctx, layout, copies, total_steps, first_step=0, chunk=512):
    """CUDA graphs that run steps first_step .. first_step+total_steps-1 (copy = step mod copies)."""
    graphs, done = [], 0
    stream = torch.cuda.Stream()
    while done < total_steps:
        n = min(chunk, total_steps - done)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(n):
                run_step(B, ctx, layout, copies[(first_step + done + i) % len(copies)])
        graphs.append(g)
        done += n
    return graphs


def time_graphs(graphs):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for g in graphs:
        g.replay()
    e1.record()
    e1.synchronize()
    return e0.elapsed_time(e1)


def time_arm(fn_step, ncopies, steps, warmup):
    """Times an arm whose step is fn_step(copy_index) through one CUDA graph of `steps` steps."""
    stream = torch.cuda.Stream()
    for i in range(max(3, warmup)):
        fn_step(i % ncopies)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        for i in range(steps):
            fn_step(i % ncopies)
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    g.replay()
    e1.record()
    e1.synchronize()
    return e0.elapsed_time(e1) / steps


def max_over_ranks(ms: float, dist, device) -> float:
    """A multi-rank time is the slowest rank's (all-reduce MAX); a single process returns its own."""
    if dist is None:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def us_per_gemv_of_job(ms_per_step: float, n_gemv: int, world: int) -> float:
    """Every rank runs its own replica of the step: the job finishes world * n_gemv GEMVs a step time."""
    return ms_per_step * 1e3 / (n_gemv * world)


def reference_arm(args, wl):
    """Times the CPU oracle as it stands: each step decodes and multiplies a bounded sample."""
    from oracle import oracle as O

    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = os.cpu_count() or 1
    m = wl.matrices[0]
    sample_rows = min(m.rows, 512)
    codes = datagen.make_codes(m.rows, m.nb, wl.seed, m.tensor_id, count=sample_rows * m.nb).numpy().astype(np.uint64)
    scale = datagen.make_row_scale(m.rows, wl.seed, m.tensor_id).numpy()[:sample_rows]
    x = datagen.make_x(m.k, m.k_padded, wl.seed, m.tensor_id).numpy()
    for _ in range(args.warmup):
        O.matvec(codes, sample_rows, m.nb, scale, datagen.GAIN, x, nthreads=cores)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        O.matvec(codes, sample_rows, m.nb, scale, datagen.GAIN, x, nthreads=cores)
    dt = (time.perf_counter() - t0) / args.steps
    blocks_per_s = sample_rows * m.nb / dt
    # scale the sample to the whole workload: seconds per block x blocks of a step / GEMVs of a step
    us_per_gemv = wl.blocks / blocks_per_s / len(wl.matrices) * 1e6
    sample = f"{sample_rows} rows of {m.name} ({sample_rows * m.nb} blocks) per step, scaled by blocks to the whole workload"
    line = {"impl": "reference", "metric": METRIC, "value": us_per_gemv, "unit": "us", "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": wl.blocks / blocks_per_s * 1e3, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"config {wl.config}: {wl.name}", "gemvs_per_step": len(wl.matrices)},
            "cpu_baseline": {"value": us_per_gemv, "unit": "us", "cores": cores, "kind": "oracle", "sample": sample,
                             "blocks_per_s": blocks_per_s},
            "e2e": {"value": us_per_gemv, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", type=int, default=1)
    ap.add_argument("--layers", type=int, default=None, help="truncate the multi-layer stacks (configs 2, 3)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-arms", action="store_true", help="skip the one-hot / FP16 / no-weights comparison arms")
    ap.add_argument("--no-verify", action="store_true", help="skip the oracle check (profiling runs only)")
    ap.add_argument("--lean", action="store_true", help="profiling runs: no clock ramp, no end-to-end leg, no arms, no oracle check")
    ap.add_argument("--no-pdl", action="store_true", help="launch the GEMV without programmatic dependent launch")
    ap.add_argument("--ungrouped", action="store_true", help="one launch a matrix instead of row-concatenated groups")
    ap.add_argument("--profile-batch", type=int, default=0,
                    help="profiling runs: only launch llvq_gemv_batch with this many activation vectors, one launch a matrix, and exit")
    ap.add_argument("--profile-rotated", action="store_true",
                    help="profiling runs: only launch llvq_rotate and llvq_gemv_rotated on the workload's launches, and exit")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.lean:
        args.no_arms = args.no_verify = True
    wl = datagen.workload(args.config, args.layers)

    if args.impl == "reference":
        reference_arm(args, wl)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod

        dist_mod.init_process_group("nccl", device_id=device)
        dist = dist_mod

    from paper_2609_02652_b200 import binding as B, build

    build.build()
    ctx = B.create(local)
    if args.no_pdl:
        B.set_pdl(ctx, False)
    peak, peak_src = measured_peaks()

    mats = build_inputs(wl, device)
    step_bytes = sum(gemv_bytes(e["m"].rows, e["m"].nb) for e in mats)
    layout_bytes = sum(14 * e["m"].blocks for e in mats)
    ncopies = max(2, -(-3 * L2_BYTES // layout_bytes)) if layout_bytes < 3 * L2_BYTES else 1
    t0 = time.perf_counter()
    copies = make_copies(B, ctx, mats, B.PLANES, ncopies, device, grouped=not args.ungrouped)
    torch.cuda.synchronize()
    launches_per_step = len(copies[0].launches)

    if args.profile_batch:
        # a few batched launches for a profiler to capture; nothing is measured here
        nvec = args.profile_batch
        for i in range(args.warmup + args.steps):
            for ln in copies[i % ncopies].launches:
                X = ln["x"].unsqueeze(0).repeat(nvec, 1).contiguous()
                for mi, m in enumerate(ln["mats"]):
                    B.gemv_batch(ctx, ln["bufs"][mi], ln["scales"][mi], datagen.GAIN, X, m.rows, ln["k_padded"])
        torch.cuda.synchronize()
        B.status(ctx)
        print(json.dumps({"profile": "llvq_gemv_batch", "vectors": nvec, "config": wl.name, "launches": (args.warmup + args.steps) * len(mats)}))
        return

    if args.profile_rotated:
        # the rotation as a kernel of its own and inside the GEMV, for a profiler to capture; nothing is measured here
        for i in range(args.warmup + args.steps):
            for ln in copies[i % ncopies].launches:
                k = ln["mats"][0].k
                B.rotate(ctx, ln["x"][:k])
                B.gemv_rotated(ctx, ln["problems"], ln["x"], ln["k_padded"], n=k)
        torch.cuda.synchronize()
        B.status(ctx)
        print(json.dumps({"profile": "llvq_rotate + llvq_gemv_rotated", "config": wl.name,
                          "launches": 2 * (args.warmup + args.steps) * launches_per_step}))
        return

    # expander throughput (load-time step, outside the timed region)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    big = max(mats, key=lambda e: e["m"].blocks)
    B.expand(ctx, B.PLANES, big["codes"], big["m"].rows, big["m"].nb)
    e0.record()
    B.expand(ctx, B.PLANES, big["codes"], big["m"].rows, big["m"].nb)
    e1.record()
    e1.synchronize()
    expand_rate = big["m"].blocks / (e0.elapsed_time(e1) * 1e-3)

    # parity first (every row, copy 0), which also times the oracle on the host cores
    cores = os.cpu_count() or 1
    run_step(B, ctx, B.PLANES, copies[0])
    torch.cuda.synchronize()
    cpu_baseline, worst = None, None
    if not args.no_verify:
        from oracle import oracle as O

        # the multi-layer stacks are checked (and the oracle timed) on their first layer; tests/ cover more layers
        first_layer = 4 if len(mats) > 7 and not args.ungrouped else (7 if len(mats) > 7 else None)
        worst, osecs, oblocks, ogemvs = verify(O, copies, cores, first_layer)
        if rank == 0:
            cpu_baseline = {"value": osecs / ogemvs * 1e6, "unit": "us", "cores": cores, "kind": "oracle",
                            "sample": f"{ogemvs} GEMVs of the step once ({oblocks} of {wl.blocks} blocks): index decode + f64 matvec",
                            "blocks_per_s": oblocks / osecs}

    # warm-up: ramp the clocks, then W untimed steps, then exactly K timed steps
    ramp = capture_graphs(B, ctx, B.PLANES, copies, 1 if args.lean else min(512, max(64, ncopies * 8)))
    t_end = time.perf_counter() + (0.0 if args.lean else 0.4)
    while time.perf_counter() < t_end:
        time_graphs(ramp)
    warm = capture_graphs(B, ctx, B.PLANES, copies, args.warmup)
    graphs = capture_graphs(B, ctx, B.PLANES, copies, args.steps, first_step=args.warmup)
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    sampler.start()
    time_graphs(warm)
    # One untimed pass over the graphs that will be timed: a graph's first launch uploads it to the device
    # (about a millisecond for 2000 steps), which is not part of a step.  The records still rotate through
    # copies larger than L2, so the timed pass finds them cold.
    time_graphs(graphs)
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    ms = time_graphs(graphs)
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    clocks = sampler.result()
    ms = max_over_ranks(ms, dist, device)

    ms_per_step = ms / args.steps
    n_gemv = len(mats)
    us_per_gemv = us_per_gemv_of_job(ms_per_step, n_gemv, world)
    gbps = step_bytes / (ms_per_step * 1e-3) / 1e9            # per GPU
    per_shape = None

    # End to end: every step copies that step's activations from pinned host memory to the device, runs the step's
    # launches through the same C-ABI calls, copies every y back to pinned host memory and waits for it.  The
    # host buffers are one block of x and one block of y a step (the launches' vectors at 256-byte offsets), so a
    # step is one copy in, the launches, one copy out; the sequence is captured once per record copy as a CUDA
    # graph, the way a serving loop would issue it, and replayed and waited for step by step.
    def _offsets(sizes, align):
        out, at = [], 0
        for n in sizes:
            out.append(at)
            at += -(-n // align) * align
        return out, at
    l0 = copies[0].launches
    x_off, x_total = _offsets([ln["x"].numel() for ln in l0], 128)
    y_sizes = [m.rows for ln in l0 for m in ln["mats"]]
    y_off, y_total = _offsets(y_sizes, 64)
    host_x = torch.zeros(x_total, dtype=torch.float16).pin_memory()
    host_y = torch.zeros(y_total, dtype=torch.float32).pin_memory()
    dev_x = torch.zeros(x_total, dtype=torch.float16, device=device)
    dev_y = torch.zeros(y_total, dtype=torch.float32, device=device)
    for ln, off in zip(l0, x_off):
        host_x[off:off + ln["x"].numel()] = ln["x"].cpu()
    h2d = host_x.numel() * 2
    d2h = host_y.numel() * 4
    e2e_graphs = []
    e2e_keep = []
    side = torch.cuda.Stream()
    for cp in copies:
        yi = 0
        plist = []
        for ln, xo in zip(cp.launches, x_off):
            ys = []
            for m in ln["mats"]:
                ys.append(dev_y[y_off[yi]:y_off[yi] + m.rows])
                yi += 1
            plist.append((B.make_problems([(b_, s_, datagen.GAIN, y_, m.rows) for b_, s_, y_, m in zip(ln["bufs"], ln["scales"], ys, ln["mats"])]),
                          dev_x[xo:xo + ln["x"].numel()], ln["k_padded"]))
        e2e_keep.append(plist)
        def issue(plist=plist):
            dev_x.copy_(host_x, non_blocking=True)
            for probs, xv, kp in plist:
                B.gemv_grouped(ctx, B.PLANES, probs, xv, kp)
            host_y.copy_(dev_y, non_blocking=True)
        with torch.cuda.stream(side):
            issue()
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            issue()
        e2e_graphs.append(g)

    def e2e_step(i):
        e2e_graphs[i % ncopies].replay()
        torch.cuda.synchronize()

    e2e_steps = 1 if args.lean else min(args.steps, 300)
    for i in range(1 if args.lean else 10):
        e2e_step(i)
    # the copies back are the results the launches computed: the last step's y against the device arrays
    yi = 0
    for ln in copies[(0 if args.lean else 9) % ncopies].launches:
        for m in ln["mats"]:
            assert torch.equal(host_y[y_off[yi]:y_off[yi] + m.rows], dev_y[y_off[yi]:y_off[yi] + m.rows].cpu())
            yi += 1
    t1 = time.perf_counter()
    for i in range(e2e_steps):
        e2e_step(i)
    e2e_us = (time.perf_counter() - t1) / e2e_steps * 1e6 / n_gemv / world
    # ... and they are the right results: one matrix of the last step against the untimed path's y (same records, same x)
    run_step(B, ctx, B.PLANES, copies[(e2e_steps - 1) % ncopies])
    torch.cuda.synchronize()
    assert torch.equal(host_y[y_off[0]:y_off[0] + l0[0]["mats"][0].rows], copies[(e2e_steps - 1) % ncopies].launches[0]["ys"][0].cpu())

    arms = {}
    if len(mats) > 7:
        args.no_arms = True          # the comparison arms and per-shape timings are taken on the single-layer workloads
    if not args.no_arms and rank == 0:
        arm_steps = min(args.steps, 200)
        # per-matrix timings of the 14-byte-layout kernel, one launch each
        per_shape = {}
        for li, ln in enumerate(copies[0].launches):
            for mi, m in enumerate(ln["mats"]):
                def one(i, li=li, mi=mi):
                    l2 = copies[i % ncopies].launches[li]
                    B.gemv(ctx, B.PLANES, l2["bufs"][mi], l2["scales"][mi], datagen.GAIN, l2["x"], l2["mats"][mi].rows, l2["k_padded"], y=l2["ys"][mi])
                t = time_arm(one, ncopies, arm_steps, 3)
                by = gemv_bytes(m.rows, m.nb)
                per_shape[m.name] = {"rows": m.rows, "k": m.k, "us": t * 1e3, "gbps": by / (t * 1e-3) / 1e9, "frac": by / (t * 1e-3) / 1e9 / peak}
        # small-batch decode: the same matrices, one launch each, 1 / 2 / 4 activation vectors a launch (the records
        # are read and decoded once a launch; every vector was checked against the single-vector result by the tests)
        batch_arm = {}
        for nvec in (1, 2, 4):
            xb = {}
            for cp in copies:
                for ln in cp.launches:
                    if id(ln["x"]) not in xb:
                        xb[id(ln["x"])] = (ln["x"].unsqueeze(0).repeat(nvec, 1).contiguous(),
                                           [torch.empty((nvec, m.rows), dtype=torch.float32, device=device) for m in ln["mats"]])
            def bstep(i, xb=xb):
                for ln in copies[i % ncopies].launches:
                    X, Ys = xb[id(ln["x"])]
                    for mi, m in enumerate(ln["mats"]):
                        B.gemv_batch(ctx, ln["bufs"][mi], ln["scales"][mi], datagen.GAIN, X, m.rows, ln["k_padded"], y=Ys[mi])
            t = time_arm(bstep, ncopies, arm_steps, 3)
            batch_arm[str(nvec)] = {"us_per_launch": t * 1e3 / n_gemv, "us_per_vector": t * 1e3 / n_gemv / nvec,
                                    "record_gbps": step_bytes / (t * 1e-3) / 1e9}
            del xb
        arms["batch"] = batch_arm
        # activation rotation ahead of every projection (the served order: the weights live in the rotated basis, so
        # each projection's input is rotated first).  The rotation acts on the k real entries of x; the zero padding
        # passes through.  Three timings: the rotation inside the GEMV's own launch (llvq_gemv_rotated), the
        # rotation as a kernel of its own ahead of each GEMV (llvq_rotate, the paper's arrangement), and those
        # rotation kernels alone.
        xr = {}
        for cp in copies:
            for ln in cp.launches:
                if id(ln["x"]) not in xr:
                    xr[id(ln["x"])] = ln["x"].clone()
        def rot_fused(i):
            for ln in copies[i % ncopies].launches:
                B.gemv_rotated(ctx, ln["problems"], ln["x"], ln["k_padded"], n=ln["mats"][0].k)
        def rot_two(i):
            for ln in copies[i % ncopies].launches:
                k = ln["mats"][0].k
                B.rotate(ctx, ln["x"][:k], y=xr[id(ln["x"])][:k])
                B.gemv_grouped(ctx, B.PLANES, ln["problems"], xr[id(ln["x"])], ln["k_padded"])
        def rot_only(i):
            for ln in copies[i % ncopies].launches:
                k = ln["mats"][0].k
                B.rotate(ctx, ln["x"][:k], y=xr[id(ln["x"])][:k])
        def rot_fused_512(i):
            for ln in copies[i % ncopies].launches:
                B.gemv_rotated(ctx, ln["problems"], ln["x"], ln["k_padded"], n=ln["mats"][0].k, block=min(512, int(B.rotate_block(ln["mats"][0].k))))
        t_f = time_arm(rot_fused, ncopies, arm_steps, 3)
        t_f512 = time_arm(rot_fused_512, ncopies, arm_steps, 3)
        t_2 = time_arm(rot_two, ncopies, arm_steps, 3)
        t_0 = time_arm(rot_only, ncopies, arm_steps, 3)
        n_launch = len(copies[0].launches)
        arms["rotated"] = {"us_per_gemv_fused": t_f * 1e3 / n_gemv, "us_per_gemv_fused_blocks_of_512_at_most": t_f512 * 1e3 / n_gemv,
                           "us_per_gemv_two_launches": t_2 * 1e3 / n_gemv,
                           "us_per_rotation_alone": t_0 * 1e3 / n_launch, "rotations_per_step": n_launch,
                           "block_lengths": sorted({int(B.rotate_block(ln["mats"][0].k)) for ln in copies[0].launches})}
        # no-weights control: the same launches without record reads
        def nw(i):
            for ln in copies[i % ncopies].launches:
                for mi, m in enumerate(ln["mats"]):
                    B.gemv_noweights(ctx, ln["scales"][mi], ln["x"], m.rows, ln["k_padded"], y=ln["ys"][mi])
        t = time_arm(nw, ncopies, arm_steps, 3)
        arms["noweights"] = {"us_per_gemv": t * 1e3 / n_gemv, "launches_per_step": n_gemv}
        # the 13-byte layout: the same codes and arithmetic, a one-byte header (exact for every block)
        p13_copies = make_copies(B, ctx, mats, B.PLANES13, ncopies, device, grouped=not args.ungrouped)
        run_step(B, ctx, B.PLANES13, p13_copies[0])
        torch.cuda.synchronize()
        run_step(B, ctx, B.PLANES, copies[0])
        torch.cuda.synchronize()
        same_outputs(copies, p13_copies, exact=True)
        t = time_arm(lambda i: run_step(B, ctx, B.PLANES13, p13_copies[i % len(p13_copies)]), len(p13_copies), arm_steps, 3)
        pb = sum(gemv_bytes(e["m"].rows, e["m"].nb, 13) for e in mats)
        arms["planes13"] = {"us_per_gemv": t * 1e3 / n_gemv, "gbps": pb / (t * 1e-3) / 1e9, "frac": pb / (t * 1e-3) / 1e9 / peak,
                            "bytes_per_block": 13, "bits_per_weight": 13 * 8 / 24}
        del p13_copies
        # one-hot layout
        oh_copies = make_copies(B, ctx, mats, B.ONEHOT, max(2, ncopies * 14 // 20 + 1), device, grouped=not args.ungrouped)
        run_step(B, ctx, B.ONEHOT, oh_copies[0])
        torch.cuda.synchronize()
        run_step(B, ctx, B.PLANES, copies[0])
        torch.cuda.synchronize()
        same_outputs(copies, oh_copies, exact=False)
        t = time_arm(lambda i: run_step(B, ctx, B.ONEHOT, oh_copies[i % len(oh_copies)]), len(oh_copies), arm_steps, 3)
        ob = sum(gemv_bytes(e["m"].rows, e["m"].nb, 20) for e in mats)
        arms["onehot"] = {"us_per_gemv": t * 1e3 / n_gemv, "gbps": ob / (t * 1e-3) / 1e9, "frac": ob / (t * 1e-3) / 1e9 / peak, "bytes_per_block": 20}
        del oh_copies
        # FP16 control over the decoded weights
        fp_copies = []
        nfp = max(2, -(-3 * L2_BYTES // (48 * sum(e["m"].blocks for e in mats))))
        for c in range(nfp):
            ws = []
            for ln in copies[0].launches:
                for mi, m in enumerate(ln["mats"]):
                    W = B.dequant_fp16(ctx, B.PLANES, ln["bufs"][mi], ln["scales"][mi], datagen.GAIN, m.rows, ln["k_padded"])
                    ws.append((W, ln["x"], m, torch.empty(m.rows, dtype=torch.float32, device=device)))
            fp_copies.append(ws)
        def fp(i):
            for W, x, m, y in fp_copies[i % nfp]:
                B.gemv_fp16(W, x, m.rows, m.k_padded, y=y)
        t = time_arm(fp, nfp, arm_steps, 3)
        fb = sum(2 * e["m"].rows * e["m"].k_padded + 2 * e["m"].k_padded + 4 * e["m"].rows for e in mats)
        arms["fp16"] = {"us_per_gemv": t * 1e3 / n_gemv, "gbps": fb / (t * 1e-3) / 1e9, "frac": fb / (t * 1e-3) / 1e9 / peak}
        arms["planes_vs_fp16"] = arms["fp16"]["us_per_gemv"] / (ms_per_step * 1e3 / n_gemv)
        del fp_copies

    if rank == 0:
        line = {
            "metric": METRIC, "value": us_per_gemv, "unit": "us", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "u8 x s8 -> s32 (tensor cores), f32 block scale, int64 row sums", "data": "synthetic",
            "config": {"workload": f"config {wl.config}: {wl.name}", "gemvs_per_step": n_gemv, "launches_per_step": launches_per_step,
                       "layout": "Planes14: 14 B per 24 weights - class, gain, 24 four-bit sign+level codes (4.67 b/w payload; the paper's 4.80 b/w label counts its f32 tail and scales)",
                       "l2": f"records and scales rotate through {ncopies} distinct copies ({ncopies * layout_bytes / 1e6:.0f} MB) so no launch finds its records in L2; x (a few KB a launch) is one buffer, as in a decoder where it is the previous operator's output",
                       "multi_gpu": "replicas only: each rank runs the whole step on its own copy", "seed": wl.seed},
            "gbps": gbps, "hbm_frac": gbps / peak, "bytes_per_step": step_bytes,
            "roofline": {"bound": "hbm", "achieved": gbps, "peak": peak, "unit": "GB/s", "frac": gbps / peak,
                         "traffic": step_bytes / launches_per_step * NCU_TRAFFIC_PER_ALGORITHMIC_BYTE,
                         "traffic_note": "DRAM bytes per launch (mean over the step's launches): ncu capture of the 8192x8192 launch scaled by bytes",
                         "kernel": "gemv_planes_kernel", "peak_source": peak_src,
                         # the competing ceiling, from the ncu capture in profiles/ (8192 x 8192 launch): instruction issue
                         "secondary": {"bound": "issue", "warp_instructions_per_block_column": NCU_WARP_INSTR_PER_CELL,
                                       "issue_slots_busy_pct": NCU_ISSUE_BUSY_PCT,
                                       "source": "profiles/gemv_planes_kernel_config4_8192x8192.txt"},
                         "how": "algorithmic bytes of a step / CUDA-event time of the step, averaged over its launches"},
            "cpu_baseline": cpu_baseline,
            "e2e": {"value": e2e_us, "unit": "us", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "how": "every step: one copy of the step's x vectors from pinned host memory, the launches, one copy of every y back to pinned host memory, issued as a captured CUDA graph of those C-ABI calls and waited for before the next step"},
            "gpu_launches": args.steps * launches_per_step,
            "clocks": clocks, "parity_worst_normalised_error": worst,
            "expand_blocks_per_s": expand_rate, "per_shape": per_shape, "arms": arms,
        }
        print(json.dumps(line), flush=True)
    ctx.close()
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
