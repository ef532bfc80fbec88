#!/usr/bin/env python
"""Benchmark of the batch-1 lattice GEMV path (one JSON line on stdout, rank 0).

A step is one pass over the workload's per-token sequence of lattice GEMVs: for the default workload, the
14B-like stack, the 280 projections of 40 decoder layers issued as 160 row-concatenated launches (q/k/v and
gate/up share a launch).  Inputs are synthetic and seeded.  Every row of the first layer of the timed path is
checked against the f64 CPU oracle before anything is timed (that check is also the cpu_baseline leg: the
oracle's time on the host cores).  The records are larger than L2 (or rotate through enough distinct copies),
so no launch finds its records there.

Protocol: W untimed warm-up steps, then `--rounds` rounds (seven unless told otherwise) of exactly K steps each,
each round bracketed by a barrier and a device synchronisation and timed with CUDA events on the launching
stream; the first two rounds are discarded, `value` is the median of the rest, `min` / `max` its range.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--rounds R] [--impl reference]

With --impl reference the CPU oracle itself is timed on the host cores (one whole GEMV of the workload a step).
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
# 8192 x 8192 launch (profiles/gemv_planes_kernel_config4_8192x8192.txt); traffic grows in proportion
# to the records streamed, so a launch's traffic is its bytes times this.
NCU_TRAFFIC_PER_ALGORITHMIC_BYTE = 39.362304 / 39.288864
# from the same capture: warp instructions per block column (32 rows x 24 weights), and the share of issue
# slots busy over the launch
NCU_WARP_INSTR_PER_CELL = 5668779 / 87552
NCU_ISSUE_BUSY_PCT = 54.4
METRIC = "us_per_lattice_gemv"
DISCARD_ROUNDS = 2


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
    """Codes (on the device), scales and x (on the host) for every matrix; x is shared inside a launch group."""
    mats = []
    group_x = {}
    for m in wl.matrices:
        key = m.group if m.group >= 0 else ("solo", m.tensor_id)
        if key not in group_x:
            group_x[key] = datagen.make_x(m.k, m.k_padded, wl.seed, m.tensor_id)
        mats.append(dict(m=m, key=key, codes=datagen.make_codes(m.rows, m.nb, wl.seed, m.tensor_id, device=device),
                         scale=datagen.make_row_scale(m.rows, wl.seed, m.tensor_id), x=group_x[key]))
    return mats


def make_copies(B, ctx, mats, layout, ncopies, device, grouped=True, keep_codes=None):
    """Expands every matrix once and clones the records ncopies - 1 times.  Codes of matrices outside
    `keep_codes` (a set of tensor ids, None = all) are dropped once expanded: they are needed only by the oracle."""
    first = {}
    for e in mats:
        m = e["m"]
        out = None
        if layout == B.PLANES10X:      # a buffer with room for exactly the matrix's exceptions
            out = torch.empty(B.overlay_bytes(m.rows, m.k_padded, B.overlay_count(ctx, e["codes"], m.rows, m.nb)), dtype=torch.uint8, device=device)
        first[m.tensor_id] = B.expand(ctx, layout, e["codes"], m.rows, m.nb, out=out)
        if keep_codes is not None and m.tensor_id not in keep_codes:
            e["codes"] = None
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


def copies_needed(layout_bytes: int) -> int:
    """Distinct copies of the records so that a launch never finds its records in L2: three times L2 in rotation."""
    return max(2, -(-3 * L2_BYTES // layout_bytes)) if layout_bytes < 3 * L2_BYTES else 1


def run_step(B, ctx, layout, cp):
    for ln in cp.launches:
        B.gemv_grouped(ctx, layout, ln["problems"], ln["x"], ln["k_padded"])


def verify(oracle, copies, threads, max_launches=None):
    """Every row of copy 0 (of its first max_launches launches) against the f64 oracle.
    Returns (worst normalised error, oracle seconds, blocks, GEMVs checked, seconds of index decode alone on one core)."""
    worst, secs, blocks, gemvs, decode_secs = 0.0, 0.0, 0, 0, 0.0
    for ln in copies[0].launches[:max_launches]:
        xh = ln["x"].cpu().numpy()
        for e, y in zip(ln["members"], ln["ys"]):
            m = e["m"]
            codes = e["codes"].cpu().numpy().astype(np.uint64)
            t0 = time.perf_counter()
            y_ref, wn, ab = oracle.matvec(codes, m.rows, m.nb, e["scale"].numpy(), datagen.GAIN, xh, nthreads=threads)
            secs += time.perf_counter() - t0
            # the decode alone, on a bounded sample of the same codes (one core), scaled to the matrix by blocks
            sample = codes.reshape(-1)[:min(codes.size, 1 << 18)]
            t0 = time.perf_counter()
            oracle.decode_batch(sample)
            decode_secs += (time.perf_counter() - t0) * (m.blocks / sample.size)
            blocks += m.blocks
            yv = y.cpu().numpy().astype(np.float64)
            denom = wn * float(np.linalg.norm(xh.astype(np.float64)))
            err = np.abs(yv - y_ref)
            ratio = np.where(denom > 0, err / np.where(denom > 0, denom, 1.0), 0.0)
            if not (np.isfinite(yv).all() and ratio.max() <= 1e-4 and (yv[denom == 0] == 0).all()):
                raise SystemExit(f"parity failure on {m.name}: normalised error {ratio.max():.3e}")
            worst = max(worst, float(ratio.max()))
            gemvs += 1
    return worst, secs, blocks, gemvs, decode_secs


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


def capture_graphs(fn_step, total_steps, first_step=0, chunk=512):
    """CUDA graphs that run fn_step(first_step) .. fn_step(first_step + total_steps - 1)."""
    graphs, done = [], 0
    stream = torch.cuda.Stream()
    while done < total_steps:
        n = min(chunk, total_steps - done)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(n):
                fn_step(first_step + done + i)
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


def summarise_rounds(ms_rounds):
    """Median and range of the rounds kept (the first DISCARD_ROUNDS are dropped when enough rounds were run)."""
    kept = ms_rounds[DISCARD_ROUNDS:] if len(ms_rounds) > DISCARD_ROUNDS else ms_rounds
    return statistics.median(kept), min(kept), max(kept), len(kept)


def time_rounds(fn_step, steps, warmup, rounds, dist=None, device=None):
    """The protocol: warm-up steps, one untimed replay of the timed graphs (a graph's first launch uploads it,
    which is not a step), then `rounds` timed replays of exactly `steps` steps, each between a barrier and a
    synchronisation; a multi-rank round counts as its slowest rank's.  Returns the list of ms per round."""
    warm = capture_graphs(fn_step, max(3, warmup))
    graphs = capture_graphs(fn_step, steps, first_step=max(3, warmup))
    torch.cuda.synchronize()
    time_graphs(warm)
    time_graphs(graphs)
    out = []
    for _ in range(rounds):
        if dist:
            dist.barrier()
        torch.cuda.synchronize()
        ms = time_graphs(graphs)
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        out.append(max_over_ranks(ms, dist, device))
    return out


def time_arm(fn_step, ncopies, steps, warmup, rounds=5):
    """Median ms per step of an arm whose step is fn_step(copy_index)."""
    med, _, _, _ = summarise_rounds([ms / steps for ms in time_rounds(lambda i: fn_step(i % ncopies), steps, warmup, rounds)])
    return med


def reference_arm(args, wl):
    """Times the CPU oracle as it stands: each step decodes and multiplies one whole GEMV of the workload (its
    smallest matrix, so that a step stays bounded); value and ms_per_step are that GEMV's measured time."""
    from oracle import oracle as O

    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = os.cpu_count() or 1
    m = min(wl.matrices, key=lambda mm: mm.blocks)
    codes = datagen.make_codes(m.rows, m.nb, wl.seed, m.tensor_id).numpy().astype(np.uint64)
    scale = datagen.make_row_scale(m.rows, wl.seed, m.tensor_id).numpy()
    x = datagen.make_x(m.k, m.k_padded, wl.seed, m.tensor_id).numpy()
    for _ in range(args.warmup):
        O.matvec(codes, m.rows, m.nb, scale, datagen.GAIN, x, nthreads=cores)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        O.matvec(codes, m.rows, m.nb, scale, datagen.GAIN, x, nthreads=cores)
    dt = (time.perf_counter() - t0) / args.steps
    sample = f"one GEMV a step: {m.name} ({m.rows} x {m.k}, {m.blocks} blocks) of {wl.name}, index decode + f64 matvec"
    line = {"impl": "reference", "metric": METRIC, "value": dt * 1e6, "unit": "us", "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"config {wl.config}: {wl.name}", "sample": sample, "gemvs_per_step": 1},
            "cpu_baseline": {"value": dt * 1e6, "unit": "us", "cores": cores, "kind": "oracle", "sample": sample,
                             "blocks_per_s": m.blocks / dt},
            "e2e": {"value": dt * 1e6, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def figures(ms_per_step, n_gemv, step_bytes, peak):
    gbps = step_bytes / (ms_per_step * 1e-3) / 1e9
    return {"us": ms_per_step * 1e3 / n_gemv, "gbps": gbps, "frac": gbps / peak}


def side_workload(B, ctx, config, device, peak, steps_target=3000, rounds=7):
    """Another configuration through the same protocol (no oracle run here: the GPU tests check these workloads)."""
    wl = datagen.workload(config)
    mats = build_inputs(wl, device)
    step_bytes = sum(gemv_bytes(e["m"].rows, e["m"].nb) for e in mats)
    layout_bytes = sum(14 * e["m"].blocks for e in mats)
    ncopies = copies_needed(layout_bytes)
    copies = make_copies(B, ctx, mats, B.PLANES, ncopies, device, keep_codes=set())
    launches = len(copies[0].launches)
    steps = max(3, min(400, steps_target // launches))
    med, lo, hi, kept = summarise_rounds([ms / steps for ms in time_rounds(lambda i: run_step(B, ctx, B.PLANES, copies[i % ncopies]),
                                                                           steps, 3, rounds)])
    B.status(ctx)
    out = figures(med, len(mats), step_bytes, peak)
    out.update({"workload": f"config {config}: {wl.name}", "us_min": lo * 1e3 / len(mats), "us_max": hi * 1e3 / len(mats),
                "gemvs_per_step": len(mats), "launches_per_step": launches, "steps": steps, "rounds_kept": kept,
                "bytes_per_step": step_bytes, "record_copies": ncopies})
    del copies, mats
    torch.cuda.empty_cache()
    return out


def single_matrix(B, ctx, rows, k, device, peak, seed=5, rounds=7, steps=200):
    """One matrix, one launch a step, cold records."""
    nb = (k + 23) // 24
    codes = datagen.make_codes(rows, nb, seed, device=device)
    sc = datagen.make_row_scale(rows, seed).to(device)
    x = datagen.make_x(k, nb * 24, seed).to(device)
    buf0 = B.expand(ctx, B.PLANES, codes, rows, nb)
    del codes
    ncopies = copies_needed(buf0.numel())
    bufs = [buf0] + [buf0.clone() for _ in range(ncopies - 1)]
    y = torch.empty(rows, dtype=torch.float32, device=device)
    med, lo, hi, _ = summarise_rounds([ms / steps for ms in time_rounds(
        lambda i: B.gemv(ctx, B.PLANES, bufs[i % ncopies], sc, datagen.GAIN, x, rows, nb * 24, y=y), steps, 3, rounds)])
    nw, _, _, _ = summarise_rounds([ms / steps for ms in time_rounds(
        lambda i: B.gemv_noweights(ctx, sc, x, rows, nb * 24, y=y), steps, 3, 5)])
    out = figures(med, 1, gemv_bytes(rows, nb), peak)
    out.update({"rows": rows, "k": k, "us_min": lo * 1e3, "us_max": hi * 1e3, "noweights_us": nw * 1e3})
    del bufs, buf0
    torch.cuda.empty_cache()
    return out


def overlay_used_bytes(B, ctx, mats):
    """Bytes a step reads in the 10-byte layout (short records, index, the table entries in use, scales, x, y), the
    blocks it covers and how many of them are in the exception tables."""
    used, blocks, exc = 0, 0, 0
    for e in mats:
        m = e["m"]
        n = B.overlay_count(ctx, e["codes"], m.rows, m.nb)
        used += B.overlay_bytes(m.rows, m.k_padded, n) + gemv_bytes(m.rows, m.nb, 0)
        blocks += m.blocks
        exc += n
    return used, blocks, exc


def with_exceptions(B, ctx, e, share, seed):
    """The matrix's code words with a share of the blocks replaced by exception blocks of the 10-byte layout, drawn from
    those the matrix itself contains (found by decoding it with the library and applying the layout's window rule)."""
    m, codes = e["m"], e["codes"]
    co, _ = B.decode_i8(ctx, B.PLANES, B.expand(ctx, B.PLANES, codes, m.rows, m.nb), m.rows, m.nb)
    u = 8 + torch.div(co.reshape(-1, 24).to(torch.int32), 2, rounding_mode="floor")
    lo, hi = u.min(1).values, u.max(1).values
    pool = codes.reshape(-1)[torch.clamp(hi - 7, min=3) > torch.clamp(lo, max=6)]
    if pool.numel() == 0:
        return codes
    g = torch.Generator(device=codes.device)
    g.manual_seed(seed)
    hit = torch.rand(codes.numel(), device=codes.device, generator=g) < share
    pick = pool[torch.randint(0, pool.numel(), (codes.numel(),), device=codes.device, generator=g)]
    return torch.where(hit, pick, codes.reshape(-1)).reshape(codes.shape)


def overlay_arm(B, ctx, mats, copies, ncopies, device, peak, steps):
    """The 10-byte layout with its exception table on the synthetic stream (about one block in eight thousand is an
    exception) and on the same matrices with 3.38 % of the blocks made exceptions (the share the paper reports for
    its own overlay on its artifact)."""
    n_gemv = len(mats)
    out = {}
    for label, share in (("synthetic_stream", None), ("exceptions_3_38_pct", 0.0338)):
        if share is None:
            ms, ref = mats, copies
        else:
            ms = [dict(e, codes=with_exceptions(B, ctx, e, share, 1000 + e["m"].tensor_id)) for e in mats]
            ref = make_copies(B, ctx, ms, B.PLANES, 1, device)
            run_step(B, ctx, B.PLANES, ref[0])
        c10 = make_copies(B, ctx, ms, B.PLANES10X, ncopies, device)
        run_step(B, ctx, B.PLANES10X, c10[0])
        torch.cuda.synchronize()
        B.status(ctx)
        same_outputs(ref, c10, exact=False)
        t = time_arm(lambda i: run_step(B, ctx, B.PLANES10X, c10[i]), len(c10), steps, 3)
        used, blocks, exc = overlay_used_bytes(B, ctx, ms)
        out[label] = dict(figures(t, n_gemv, used, peak), bytes_per_block=(used - sum(gemv_bytes(e["m"].rows, e["m"].nb, 0) for e in ms)) / blocks,
                          exception_blocks=exc, exception_share=exc / blocks)
        out[label]["bits_per_weight"] = out[label]["bytes_per_block"] * 8 / 24
        del c10, ref
    return out


def comparison_arms(B, ctx, device, peak, steps=200):
    """The arms of the paper's layout table, on the 4B-like layer (config 1): per-matrix launches, small batches,
    the activation rotation, the no-weights control, the 13-byte and the 10-byte layout, the one-hot layout, the FP16 control.
    Every arm's outputs are compared with those of the 14-byte arm (which the GPU tests hold to the oracle)."""
    wl = datagen.workload(1)
    mats = build_inputs(wl, device)
    n_gemv = len(mats)
    step_bytes = sum(gemv_bytes(e["m"].rows, e["m"].nb) for e in mats)
    ncopies = copies_needed(sum(14 * e["m"].blocks for e in mats))
    copies = make_copies(B, ctx, mats, B.PLANES, ncopies, device)
    t_main = time_arm(lambda i: run_step(B, ctx, B.PLANES, copies[i]), ncopies, steps, 3)
    arms = {"workload": f"config 1: {wl.name}", "planes14": figures(t_main, n_gemv, step_bytes, peak)}
    # per-matrix timings of the 14-byte-layout kernel, one launch each
    per_matrix = {}
    for li, ln in enumerate(copies[0].launches):
        for mi, m in enumerate(ln["mats"]):
            def one(i, li=li, mi=mi):
                l2 = copies[i].launches[li]
                B.gemv(ctx, B.PLANES, l2["bufs"][mi], l2["scales"][mi], datagen.GAIN, l2["x"], l2["mats"][mi].rows, l2["k_padded"], y=l2["ys"][mi])
            t = time_arm(one, ncopies, steps, 3)
            per_matrix[m.name] = dict(figures(t, 1, gemv_bytes(m.rows, m.nb), peak), rows=m.rows, k=m.k)
    arms["per_matrix"] = per_matrix
    # small-batch decode: the same matrices, one launch each, 1 / 2 / 4 activation vectors a launch
    batch_arm = {}
    for nvec in (1, 2, 4):
        xb = {}
        for cp in copies:
            for ln in cp.launches:
                if id(ln["x"]) not in xb:
                    xb[id(ln["x"])] = (ln["x"].unsqueeze(0).repeat(nvec, 1).contiguous(),
                                       [torch.empty((nvec, m.rows), dtype=torch.float32, device=device) for m in ln["mats"]])
        def bstep(i, xb=xb):
            for ln in copies[i].launches:
                X, Ys = xb[id(ln["x"])]
                for mi, m in enumerate(ln["mats"]):
                    B.gemv_batch(ctx, ln["bufs"][mi], ln["scales"][mi], datagen.GAIN, X, m.rows, ln["k_padded"], y=Ys[mi])
        t = time_arm(bstep, ncopies, steps, 3)
        batch_arm[str(nvec)] = {"us_per_launch": t * 1e3 / n_gemv, "us_per_vector": t * 1e3 / n_gemv / nvec,
                                "record_gbps": step_bytes / (t * 1e-3) / 1e9}
        del xb
    arms["batch"] = batch_arm
    # activation rotation ahead of every projection (the served order): inside the GEMV's own launch, as a kernel
    # of its own ahead of each GEMV (the paper's arrangement), and those rotation kernels alone
    xr = {}
    for cp in copies:
        for ln in cp.launches:
            if id(ln["x"]) not in xr:
                xr[id(ln["x"])] = ln["x"].clone()
    def rot_fused(i):
        for ln in copies[i].launches:
            B.gemv_rotated(ctx, ln["problems"], ln["x"], ln["k_padded"], n=ln["mats"][0].k)
    def rot_two(i):
        for ln in copies[i].launches:
            k = ln["mats"][0].k
            B.rotate(ctx, ln["x"][:k], y=xr[id(ln["x"])][:k])
            B.gemv_grouped(ctx, B.PLANES, ln["problems"], xr[id(ln["x"])], ln["k_padded"])
    def rot_only(i):
        for ln in copies[i].launches:
            k = ln["mats"][0].k
            B.rotate(ctx, ln["x"][:k], y=xr[id(ln["x"])][:k])
    def rot_fused_512(i):
        for ln in copies[i].launches:
            B.gemv_rotated(ctx, ln["problems"], ln["x"], ln["k_padded"], n=ln["mats"][0].k, block=min(512, int(B.rotate_block(ln["mats"][0].k))))
    n_launch = len(copies[0].launches)
    arms["rotated"] = {"us_per_gemv_fused": time_arm(rot_fused, ncopies, steps, 3) * 1e3 / n_gemv,
                       "us_per_gemv_fused_blocks_of_512_at_most": time_arm(rot_fused_512, ncopies, steps, 3) * 1e3 / n_gemv,
                       "us_per_gemv_two_launches": time_arm(rot_two, ncopies, steps, 3) * 1e3 / n_gemv,
                       "us_per_rotation_alone": time_arm(rot_only, ncopies, steps, 3) * 1e3 / n_launch, "rotations_per_step": n_launch,
                       "block_lengths": sorted({int(B.rotate_block(ln["mats"][0].k)) for ln in copies[0].launches})}
    # no-weights control: the same launches without record reads
    def nw(i):
        for ln in copies[i].launches:
            for mi, m in enumerate(ln["mats"]):
                B.gemv_noweights(ctx, ln["scales"][mi], ln["x"], m.rows, ln["k_padded"], y=ln["ys"][mi])
    arms["noweights"] = {"us_per_gemv": time_arm(nw, ncopies, steps, 3) * 1e3 / n_gemv, "launches_per_step": n_gemv}
    # the 13-byte layout: the same codes and arithmetic, a one-byte header (exact for every block)
    run_step(B, ctx, B.PLANES, copies[0])
    p13_copies = make_copies(B, ctx, mats, B.PLANES13, ncopies, device)
    run_step(B, ctx, B.PLANES13, p13_copies[0])
    torch.cuda.synchronize()
    same_outputs(copies, p13_copies, exact=True)
    t = time_arm(lambda i: run_step(B, ctx, B.PLANES13, p13_copies[i]), len(p13_copies), steps, 3)
    pb = sum(gemv_bytes(e["m"].rows, e["m"].nb, 13) for e in mats)
    arms["planes13"] = dict(figures(t, n_gemv, pb, peak), bytes_per_block=13, bits_per_weight=13 * 8 / 24)
    del p13_copies
    # the 10-byte layout: three-bit window codes, the blocks no window holds kept exactly in a table (the sparse overlay)
    arms["planes10x"] = overlay_arm(B, ctx, mats, copies, ncopies, device, peak, steps)
    # one-hot layout: a correctness reference for the paper's other record (plain coalesced loads, scalar
    # arithmetic, not tuned), so its time says nothing about the layouts' relative merit
    oh_copies = make_copies(B, ctx, mats, B.ONEHOT, max(2, ncopies * 14 // 20 + 1), device)
    run_step(B, ctx, B.ONEHOT, oh_copies[0])
    torch.cuda.synchronize()
    same_outputs(copies, oh_copies, exact=False)
    t = time_arm(lambda i: run_step(B, ctx, B.ONEHOT, oh_copies[i]), len(oh_copies), steps, 3)
    ob = sum(gemv_bytes(e["m"].rows, e["m"].nb, 20) for e in mats)
    arms["onehot"] = dict(figures(t, n_gemv, ob, peak), bytes_per_block=20,
                          note="untuned correctness reference: not a comparison of the layouts")
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
        for W, x, m, y in fp_copies[i]:
            B.gemv_fp16(W, x, m.rows, m.k_padded, y=y)
    t = time_arm(fp, nfp, steps, 3)
    fb = sum(2 * e["m"].rows * e["m"].k_padded + 2 * e["m"].k_padded + 4 * e["m"].rows for e in mats)
    arms["fp16"] = figures(t, n_gemv, fb, peak)
    arms["planes_vs_fp16"] = arms["fp16"]["us"] / arms["planes14"]["us"]
    B.status(ctx)
    del fp_copies, copies, mats
    torch.cuda.empty_cache()
    return arms


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--rounds", type=int, default=7, help="timed rounds of --steps steps each; the first two are discarded")
    ap.add_argument("--config", type=int, default=3)
    ap.add_argument("--layers", type=int, default=None, help="truncate the multi-layer stacks (configs 2, 3)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-arms", action="store_true", help="skip the other configurations, the single matrices and the comparison arms")
    ap.add_argument("--no-pdl", action="store_true", help="launch the GEMV without programmatic dependent launch")
    ap.add_argument("--ungrouped", action="store_true", help="one launch a matrix instead of row-concatenated groups")
    ap.add_argument("--layout", default="planes14", choices=["planes14", "planes10x"], help="record layout of the timed step (the headline is planes14)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    args.rounds = max(args.rounds, DISCARD_ROUNDS + 1)
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
    n_gemv = len(mats)
    L = B.PLANES10X if args.layout == "planes10x" else B.PLANES
    if L == B.PLANES:
        step_bytes = sum(gemv_bytes(e["m"].rows, e["m"].nb) for e in mats)
        layout_bytes = sum(14 * e["m"].blocks for e in mats)
    else:
        step_bytes, _, _ = overlay_used_bytes(B, ctx, mats)
        layout_bytes = sum(10 * e["m"].blocks for e in mats)
    ncopies = copies_needed(layout_bytes)
    # the oracle checks the first layer (the multi-layer stacks) or the whole step: only those codes are kept
    checked = 7 if n_gemv > 7 else n_gemv
    copies = make_copies(B, ctx, mats, L, ncopies, device, grouped=not args.ungrouped,
                         keep_codes={e["m"].tensor_id for e in mats[:checked]})
    torch.cuda.synchronize()
    launches_per_step = len(copies[0].launches)

    # expander throughput (load-time step, outside the timed region)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    big = max(mats[:checked], key=lambda e: e["m"].blocks)
    B.expand(ctx, L, big["codes"], big["m"].rows, big["m"].nb)
    e0.record()
    B.expand(ctx, L, big["codes"], big["m"].rows, big["m"].nb)
    e1.record()
    e1.synchronize()
    expand_rate = big["m"].blocks / (e0.elapsed_time(e1) * 1e-3)

    # parity first (every row of the checked launches, copy 0), which also times the oracle on the host cores
    cores = os.cpu_count() or 1
    run_step(B, ctx, L, copies[0])
    torch.cuda.synchronize()
    from oracle import oracle as O

    checked_launches = None if checked == n_gemv else (4 if not args.ungrouped else 7)
    worst, osecs, oblocks, ogemvs, dsecs = verify(O, copies, cores, checked_launches)
    cpu_baseline = None
    if rank == 0:
        decode_us = dsecs / cores / ogemvs * 1e6
        cpu_baseline = {"value": osecs / ogemvs * 1e6, "unit": "us", "cores": cores, "kind": "oracle",
                        "sample": f"{ogemvs} GEMVs of the step once ({oblocks} of {wl.blocks} blocks): index decode + f64 matvec on all cores",
                        "blocks_per_s": oblocks / osecs, "decode_us": decode_us, "matvec_us": max(osecs / ogemvs * 1e6 - decode_us, 0.0),
                        "split": "decode_us = the index decode alone timed on one core over 262144 codes a matrix, scaled by blocks and divided by the cores; matvec_us = the rest"}

    # warm-up: ramp the clocks, then the protocol
    step_fn = lambda i: run_step(B, ctx, L, copies[i % ncopies])
    ramp = capture_graphs(step_fn, max(2, min(64, 4000 // launches_per_step)))
    t_end = time.perf_counter() + 0.4
    while time.perf_counter() < t_end:
        time_graphs(ramp)
    del ramp
    sampler = ClockSampler(local)
    sampler.start()
    ms_rounds = time_rounds(step_fn, args.steps, args.warmup, args.rounds, dist, device)
    clocks = sampler.result()
    B.status(ctx)
    ms, ms_min, ms_max, kept = summarise_rounds(ms_rounds)
    ms_per_step = ms / args.steps
    us_per_gemv = us_per_gemv_of_job(ms_per_step, n_gemv, world)
    gbps = step_bytes / (ms_per_step * 1e-3) / 1e9            # per GPU

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
                B.gemv_grouped(ctx, L, probs, xv, kp)
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

    e2e_steps = max(3, min(args.steps, 300))
    for i in range(5):
        e2e_step(i)
    # the copies back are the results the launches computed: the last step's y against the device arrays
    yi = 0
    for ln in copies[4 % ncopies].launches:
        for m in ln["mats"]:
            assert torch.equal(host_y[y_off[yi]:y_off[yi] + m.rows], dev_y[y_off[yi]:y_off[yi] + m.rows].cpu())
            yi += 1
    e2e_rounds = []
    for _ in range(args.rounds):
        t1 = time.perf_counter()
        for i in range(e2e_steps):
            e2e_step(i)
        e2e_rounds.append((time.perf_counter() - t1) / e2e_steps * 1e6 / n_gemv / world)
    e2e_us, e2e_min, e2e_max, _ = summarise_rounds(e2e_rounds)
    # ... and they are the right results: one matrix of the last step against the untimed path's y (same records, same x)
    run_step(B, ctx, L, copies[(e2e_steps - 1) % ncopies])
    torch.cuda.synchronize()
    assert torch.equal(host_y[y_off[0]:y_off[0] + l0[0]["mats"][0].rows], copies[(e2e_steps - 1) % ncopies].launches[0]["ys"][0].cpu())
    del e2e_graphs, e2e_keep

    per_config, per_shape, arms = None, None, None
    if not args.no_arms and rank == 0 and world == 1:
        # the other configurations and three single matrices through the same protocol, then the comparison arms
        del copies, mats
        torch.cuda.empty_cache()
        per_config = {str(c): side_workload(B, ctx, c, device, peak) for c in (0, 1, 2, 4) if c != args.config}
        per_shape = {f"{r}x{k}": single_matrix(B, ctx, r, k, device, peak) for r, k in ((4096, 4096), (8192, 8192), (24576, 4096))}
        arms = comparison_arms(B, ctx, device, peak)

    if rank == 0:
        line = {
            "metric": METRIC, "value": us_per_gemv, "unit": "us", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "u8 x s8 -> s32 (tensor cores), f32 block scale, int64 row sums", "data": "synthetic",
            "config": {"workload": f"config {wl.config}: {wl.name}", "gemvs_per_step": n_gemv, "launches_per_step": launches_per_step,
                       "layout": "Planes14: 14 B per 24 weights - class, gain, 24 four-bit sign+level codes (4.67 b/w payload; the paper's 4.80 b/w label counts its f32 tail and scales)"
                                 if L == B.PLANES else "Planes10x: 10 B per 24 weights - one header byte, 24 three-bit window codes - plus the exact records of the blocks no window holds",
                       "l2": f"records and scales: {ncopies} distinct cop{'y' if ncopies == 1 else 'ies'} ({ncopies * layout_bytes / 1e6:.0f} MB, at least three times L2) so no launch finds its records in L2; x (a few KB a launch) is one buffer, as in a decoder where it is the previous operator's output",
                       "multi_gpu": "replicas only: each rank runs the whole step on its own copy", "seed": wl.seed,
                       "oracle_check": f"every row of the first {ogemvs} GEMVs before timing"},
            "rounds": {"run": len(ms_rounds), "discarded": len(ms_rounds) - kept, "statistic": "median of the rounds kept",
                       "us_min": us_per_gemv_of_job(ms_min / args.steps, n_gemv, world), "us_max": us_per_gemv_of_job(ms_max / args.steps, n_gemv, world),
                       "ms_per_round": ms_rounds},
            "gbps": gbps, "hbm_frac": gbps / peak, "bytes_per_step": step_bytes,
            "roofline": {"bound": "hbm", "achieved": gbps, "peak": peak, "unit": "GB/s", "frac": gbps / peak,
                         "traffic": step_bytes / launches_per_step * NCU_TRAFFIC_PER_ALGORITHMIC_BYTE if L == B.PLANES else None,
                         "traffic_note": "DRAM bytes per launch (mean over the step's launches): ncu capture of the 8192x8192 launch scaled by bytes",
                         "kernel": "gemv_planes_kernel", "peak_source": peak_src,
                         # the competing ceiling, from the ncu capture in profiles/ (8192 x 8192 launch): instruction issue
                         "secondary": {"bound": "issue", "warp_instructions_per_block_column": NCU_WARP_INSTR_PER_CELL,
                                       "issue_slots_busy_pct": NCU_ISSUE_BUSY_PCT,
                                       "source": "profiles/gemv_planes_kernel_config4_8192x8192.txt"},
                         "how": "algorithmic bytes of a step / median CUDA-event time of a step, averaged over its launches"},
            "cpu_baseline": cpu_baseline,
            "e2e": {"value": e2e_us, "unit": "us", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "us_min": e2e_min, "us_max": e2e_max,
                    "how": "every step: one copy of the step's x vectors from pinned host memory, the launches, one copy of every y back to pinned host memory, issued as a captured CUDA graph of those C-ABI calls and waited for before the next step"},
            "gpu_launches": args.steps * launches_per_step,
            "clocks": clocks, "parity_worst_normalised_error": worst,
            "expand_blocks_per_s": expand_rate, "per_config": per_config, "per_shape": per_shape, "arms": arms,
        }
        print(json.dumps(line), flush=True)
    ctx.close()
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
