#!/usr/bin/env python
"""Benchmark of the ZCCL hot path on B200: `python bench.py --gpus N --steps K --warmup W [--impl reference]`.

One step = one pass of the whole hot path over one 64 MiB batch (a 256^3 fp32 Fourier-mode field, the paper's
3-D scientific-field workload shape) at a value-range-relative bound of 1e-3:
  compress (range pass + bound resolution + encode), decompress, fused decompress-add-recompress against a
  second field, an emulated 8-rank ring Allreduce (each rank one eighth of the batch) and an emulated 8-rank ring
  Allgather (each rank 1 MiB).
`value` = uncompressed bytes that pass through a codec kernel per step / step time (GB/s), summed over ranks.
With N > 1 every rank runs the same step on its own differently seeded batch (independent replicas; the path has no
cross-GPU exchange).  `--impl reference` times the CPU oracle on the same step.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

SIDE = 256
N_ELEMS = SIDE ** 3                 # 2^24 elements = 64 MiB
REL = 1e-3
RANKS = 8
AG_PER_RANK = 1 << 18               # allgather: 1 MiB per rank
ROT = 4                             # rotating buffer sets, each larger than L2
MIN_TIMED_MS = 500.0                # the timed region lasts at least this long (steps are replayed to get there)
# dram__bytes_read.sum + dram__bytes_write.sum of one 64 MiB call of the fused hop (its two launches together), from an
# ncu capture of this workload: 78.5 MB read + 4.4 MB written by the hop kernel, 0.3 MB by the placement (the encoded
# rounds wait in L2 between the two, and most of the 12 MB output stream is still there when the call ends)
DRAM_TRAFFIC_FUSED_64MIB = 83.2e6
# smsp__inst_executed.sum x 32 / 2^24 of the hop kernel with both operands compressed (64 MiB, cfg1), from an ncu capture
# (31 345 480 warp-instructions per launch)
HOP_C2_INSTR_PER_ELEMENT = 59.8
METRIC = "compress / decompress / fused decomp-reduce-comp GB/s (uncompressed bytes through the codec per step)"
WORKLOAD = ("cfg1: 256^3 fp32 Fourier-mode field (64 MiB), REL 1e-3; step = compress + decompress + fused hop + "
            "8-rank ring allreduce (8 MiB/rank) + 8-rank allgather (1 MiB/rank)")


def step_units_bytes() -> dict:
    """Uncompressed bytes entering an encoder or leaving a decoder, per op of one step."""
    full = 4 * N_ELEMS
    per_rank = full // RANKS
    chunk = per_rank // RANKS
    ar = RANKS * chunk + (RANKS - 1) * RANKS * chunk + RANKS * (RANKS - 1) * chunk
    ag = RANKS * 4 * AG_PER_RANK + RANKS * (RANKS - 1) * 4 * AG_PER_RANK
    return {"compress": full, "decompress": full, "fused": full, "allreduce": ar, "allgather": ag}


def max_over_ranks(value: float, device="cpu") -> float:
    """Slowest rank's time: the job is as slow as its slowest replica."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbs(bytes_per_rank_step: float, world: int, ms_per_step: float) -> float:
    """Aggregate throughput of `world` replicas that each process bytes_per_rank_step in ms_per_step."""
    return world * bytes_per_rank_step / (ms_per_step * 1e-3) / 1e9


def make_fields(rank: int):
    from paper_2502_18554_b200 import fields
    x = fields.fourier_field_3d(SIDE, seed=1 + 10 * rank)
    loc = fields.fourier_field_3d(SIDE, seed=2 + 10 * rank)
    return x, loc


# --------------------------------------------------------------------------------------------- clocks

class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons, power = [], [], set(), []
        for ln in out.splitlines():
            f = [t.strip() for t in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------------------------- CPU oracle legs

def oracle_step(x, loc, sample_elems: int):
    """The same step on the CPU oracle, on the first `sample_elems` elements of the batch."""
    import oracle
    xs, ls = x[:sample_elems], loc[:sample_elems]
    st, _ = oracle.compress(xs, oracle.EB_REL, REL)
    oracle.decompress(st)
    oracle.drc(st, local=ls)
    per = sample_elems // RANKS
    oracle.sim_allreduce([xs[r * per:(r + 1) * per] for r in range(RANKS)], oracle.EB_REL, REL)
    ag = min(AG_PER_RANK, per)
    oracle.sim_allgather([xs[r * ag:(r + 1) * ag] for r in range(RANKS)], oracle.EB_REL, REL)
    units = step_units_bytes()
    scale = sample_elems / N_ELEMS
    total = (units["compress"] + units["decompress"] + units["fused"] + units["allreduce"]) * scale
    total += RANKS * 4 * ag + RANKS * (RANKS - 1) * 4 * ag
    return total


def run_oracle(x, loc, steps: int, warmup: int, sample_elems: int):
    for _ in range(warmup):
        oracle_step(x, loc, sample_elems)
    t0 = time.perf_counter()
    nbytes = 0
    for _ in range(steps):
        nbytes += oracle_step(x, loc, sample_elems)
    dt = time.perf_counter() - t0
    return nbytes / dt / 1e9, dt / steps * 1e3


def reference_arm(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    x, loc = make_fields(0)
    sample = N_ELEMS // 4
    gbs, ms = run_oracle(x, loc, args.steps, max(args.warmup, 1), sample)
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic", "config": {"workload": WORKLOAD},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": 1, "kind": "oracle",
                         "sample": f"first {sample} of {N_ELEMS} elements of the batch per step (one quarter)"},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------- per-config table

L2_BYTES = 126 << 20


def _timed(fn, sets: int, warmup: int = 10, iters: int = 10):
    """Mean and best device time (us) of one call fn(set index), over `iters` timed replays after `warmup`.  One
    replay is a CUDA graph of `sets` calls, one per buffer set, so that the device never waits for the host between
    calls (the entry points only enqueue); its time is divided by `sets`."""
    import torch
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for i in range(sets):
            fn(i)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(sets):
            fn(i)
    for _ in range(warmup):
        g.replay()
    torch.cuda.synchronize()
    ts = []
    for _ in range(iters):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        g.replay()
        b.record()
        b.synchronize()
        ts.append(a.elapsed_time(b) * 1e3 / sets)
    return statistics.mean(ts), min(ts)


def _timed_long(fn, sets: int, device_index: int, min_ms: float = 400.0, min_launches: int = 200, warmup: int = 3):
    """Device time (us) of one call fn(set index) over a long run: a CUDA graph of `sets` calls is replayed until
    at least `min_launches` calls and `min_ms` milliseconds have gone by, inside ONE pair of events, with the SM clock
    sampled meanwhile.  Returns (us per call, calls, median SM MHz or None)."""
    import torch
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for i in range(sets):
            fn(i)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(sets):
            fn(i)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(warmup):
        g.replay()
    b.record()
    b.synchronize()
    est_ms = max(a.elapsed_time(b) / warmup, 1e-3)
    replays = max(-(-min_launches // sets), int(min_ms / est_ms) + 1)
    sampler = ClockSampler(device_index)
    sampler.start()
    time.sleep(0.25)            # the sampler's first line takes this long to come
    a.record()
    for _ in range(replays):
        g.replay()
    b.record()
    b.synchronize()
    clocks = sampler.stop()
    return a.elapsed_time(b) * 1e3 / (replays * sets), replays * sets, clocks.get("sm_mhz")


def _codec_row(z, ctx, name, x_h, mode, eb, with_oracle: bool, loc_h=None):
    """Compress and decompress (and, with loc_h, the fused hop) of one array: time, GB/s of uncompressed bytes,
    ratio; inputs and outputs rotate over enough copies to exceed L2 several times (arrays of 256 MiB and more are
    used in place)."""
    import torch
    n = x_h.size
    nbytes = 4 * n
    sets = 1 if nbytes >= (256 << 20) else max(2, min(32, -(-4 * L2_BYTES // max(3 * nbytes // 2, 1))))
    cap = z.compress_bound(n)
    xs = [torch.from_numpy(x_h).cuda() for _ in range(sets)]
    outs = [torch.empty(cap, dtype=torch.uint8, device="cuda") for _ in range(sets)]
    ys = [torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(sets)]
    sz = torch.zeros(1, dtype=torch.int64, device="cuda")
    c_mean, c_best = _timed(lambda i: ctx.compress(xs[i], mode, eb, outs[i], sz), sets)
    rc = ctx.check()
    cbytes = int(sz.item())
    d_mean, d_best = _timed(lambda i: ctx.decompress(outs[i][:cbytes], ys[i]), sets)
    ctx.check()
    err = float((ys[0].double() - xs[0].double()).abs().max().item())
    hist = torch.zeros(33, dtype=torch.int64, device="cuda")
    ctx.stream_stats(outs[0][:cbytes], hist)
    ctx.check()
    hh = hist.cpu().numpy().astype(np.float64)
    row = {"config": name, "n": n, "bytes": nbytes, "bound": ("REL " if mode == z.EB_REL else "ABS ") + f"{eb:g}",
           "ratio": round(nbytes / cbytes, 3), "status": rc, "max_abs_err": err, "buffer_sets": sets,
           "constant_block_pct": round(100.0 * hh[0] / max(hh[32], 1.0), 2),
           "mean_code_length": round(float((hh[:32] * np.arange(32)).sum() / max(hh[32], 1.0)), 3),
           "compress_us_mean": round(c_mean, 2), "compress_us_best": round(c_best, 2),
           "compress_gbs": round(nbytes / c_mean / 1e3, 1),
           "decompress_us_mean": round(d_mean, 2), "decompress_us_best": round(d_best, 2),
           "decompress_gbs": round(nbytes / d_mean / 1e3, 1)}
    if loc_h is not None:
        locs = [torch.from_numpy(loc_h).cuda() for _ in range(sets)]
        fouts = [torch.empty(cap, dtype=torch.uint8, device="cuda") for _ in range(sets)]
        f_mean, f_best = _timed(lambda i: ctx.decompress_reduce_compress(outs[i][:cbytes], n, fouts[i], sz,
                                                                         local=locs[i]), sets)
        ctx.check()
        row.update({"fused_us_mean": round(f_mean, 2), "fused_us_best": round(f_best, 2),
                    "fused_gbs": round(nbytes / f_mean / 1e3, 1), "fused_out_ratio": round(nbytes / int(sz.item()), 3)})
        del locs, fouts
    if with_oracle:
        import oracle
        best_c = best_d = float("inf")
        for _ in range(1 if nbytes >= (1 << 30) else 3):
            t0 = time.perf_counter()
            st, _ = oracle.compress(x_h, oracle.EB_REL if mode == z.EB_REL else oracle.EB_ABS, eb)
            t1 = time.perf_counter()
            oracle.decompress(st)
            t2 = time.perf_counter()
            best_c, best_d = min(best_c, t1 - t0), min(best_d, t2 - t1)
        row["oracle_compress_gbs"] = round(nbytes / best_c / 1e9, 3)
        row["oracle_decompress_gbs"] = round(nbytes / best_d / 1e9, 3)
        row["oracle_threads"] = 1
    del xs, outs, ys
    torch.cuda.empty_cache()
    return row


def _tiled_row(z, ctx, name, x_h, mode, eb, tile):
    """Compress and decompress at another tile size (same protocol as _codec_row)."""
    import torch
    n = x_h.size
    nbytes = 4 * n
    sets = max(2, min(32, -(-4 * L2_BYTES // max(3 * nbytes // 2, 1))))
    cap = z.compress_bound_tiled(n, tile)
    xs = [torch.from_numpy(x_h).cuda() for _ in range(sets)]
    outs = [torch.empty(cap, dtype=torch.uint8, device="cuda") for _ in range(sets)]
    ys = [torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(sets)]
    sz = torch.zeros(1, dtype=torch.int64, device="cuda")
    c_mean, c_best = _timed(lambda i: ctx.compress_tiled(xs[i], mode, eb, tile, outs[i], sz), sets)
    rc = ctx.check()
    cbytes = int(sz.item())
    d_mean, d_best = _timed(lambda i: ctx.decompress_tiled(outs[i][:cbytes], tile, ys[i]), sets)
    ctx.check()
    return {"config": name, "tile": tile, "n": n, "bytes": nbytes, "bound": ("REL " if mode == z.EB_REL else "ABS ") + f"{eb:g}",
            "ratio": round(nbytes / cbytes, 3), "status": rc, "buffer_sets": sets,
            "max_abs_err": float((ys[0].double() - xs[0].double()).abs().max().item()),
            "compress_us_mean": round(c_mean, 2), "compress_us_best": round(c_best, 2),
            "compress_gbs": round(nbytes / c_mean / 1e3, 1),
            "decompress_us_mean": round(d_mean, 2), "decompress_us_best": round(d_best, 2),
            "decompress_gbs": round(nbytes / d_mean / 1e3, 1)}


def config_table(args):
    """Timings of the workload configurations 0-4 (10 warm-up + 10 timed calls each, mean and best): one JSON line
    per row on stdout.  Not part of the default run."""
    import torch
    from paper_2502_18554_b200 import build, fields, zccl as z
    if not torch.cuda.is_available():
        raise SystemExit("bench.py --table needs a CUDA device")
    build.build()
    if not args.no_cpu_baseline:
        import oracle
        oracle.build()
    orc = not args.no_cpu_baseline
    want = set(args.rows.split(","))
    emit = lambda row: print(json.dumps(row), flush=True)
    emit({"table": "configs 0-4", "host_cores": os.cpu_count(),
          "protocol": "10 warm-up + 10 timed CUDA-graph replays of one call per buffer set, CUDA events, per call"})
    big = z.Context(1 << 29, 1)

    if "cfg0" in want:
        emit(_codec_row(z, big, "cfg0", fields.smooth_1d(1 << 20, seed=0), z.EB_REL, 1e-3, orc))
    if "cfg1" in want:
        x1, loc1 = fields.fourier_field_3d(SIDE, seed=1), fields.fourier_field_3d(SIDE, seed=2)
        for eb in (1e-2, 1e-3, 1e-4):
            emit(_codec_row(z, big, "cfg1", x1, z.EB_REL, eb, orc and eb == 1e-3, loc1))
        emit(_tiled_row(z, big, "cfg1, tile of 5120", x1, z.EB_REL, 1e-3, 5120))
    if "cfg3" in want:
        emit(_codec_row(z, big, "cfg3", fields.gradient_like(1 << 28, seed=3), z.EB_ABS, 1e-5, orc))

    # cfg4: message sizes 4 KiB ... 1 GiB in steps of x4, and 2 GiB; prefixes of one cfg0-style field
    x4 = fields.smooth_1d(1 << 29 if "cfg4" in want else 1 << 27, seed=0) if want & {"cfg4", "collectives"} else None
    if "cfg4" in want:
        for log2b in list(range(12, 31, 2)) + [31]:
            for eb in ((1e-2, 1e-3, 1e-4) if log2b in (20, 26) else (1e-3,)):
                emit(_codec_row(z, big, f"cfg4 2^{log2b} B", x4[: 1 << (log2b - 2)], z.EB_REL, eb, False))
    big.close()
    torch.cuda.empty_cache()

    # cfg4 collectives: 8-rank Allgather and Bcast per message size (per-rank size up to 64 MiB)
    N = RANKS
    ctx = z.Context(1 << 27, N)
    for log2b in range(12, 27, 2) if "collectives" in want else ():
        n = 1 << (log2b - 2)
        send = [torch.from_numpy(x4[r * n:(r + 1) * n]).cuda() for r in range(N)]
        recv = [torch.empty(N * n, dtype=torch.float32, device="cuda") for _ in range(N)]
        ag_mean, ag_best = _timed(lambda i: ctx.sim_allgather(send, recv, z.EB_REL, REL), 1)
        sizes = ctx.sim_sizes()
        brecv = [torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(N)]
        bc_mean, bc_best = _timed(lambda i: ctx.sim_bcast(send[0], brecv, z.EB_REL, REL), 1)
        ctx.check()
        emit({"config": f"cfg4 collectives 2^{log2b} B per rank", "ranks": N, "bound": "REL 0.001",
              "allgather_us_mean": round(ag_mean, 2), "allgather_us_best": round(ag_best, 2),
              "allgather_gbs": round((N * 4 * n + N * (N - 1) * 4 * n) / ag_mean / 1e3, 1),
              "allgather_ratio": round(N * 4 * n / sum(sizes[:N]), 3),
              "bcast_us_mean": round(bc_mean, 2), "bcast_us_best": round(bc_best, 2),
              "bcast_gbs": round((4 * n + N * 4 * n) / bc_mean / 1e3, 1)})
        del send, recv, brecv
    del x4
    torch.cuda.empty_cache()

    if "cfg2" not in want:
        return
    # cfg2: 8 ranks x 2^24, REL 1e-3 of the global range
    send_h = fields.rank_fields(N, 1 << 24, base_seed=100)
    send = [torch.from_numpy(a).cuda() for a in send_h]
    recv = [torch.empty(1 << 24, dtype=torch.float32, device="cuda") for _ in range(N)]
    ar_mean, ar_best = _timed(lambda i: ctx.sim_allreduce(send, recv, z.EB_REL, REL), 1)
    rc = ctx.check()
    sizes = ctx.sim_sizes()
    exact = torch.zeros(1 << 24, dtype=torch.float64, device="cuda")
    for t in send:
        exact += t.double()
    err = max(float((r.double() - exact).abs().max().item()) for r in recv)
    lo = min(float(t.min().item()) for t in send)
    hi = max(float(t.max().item()) for t in send)
    chunk_bytes = 4 * (1 << 21)
    per_step = [round(N * chunk_bytes / sum(sizes[k * N:(k + 1) * N]), 3) for k in range(N)]
    units = N * chunk_bytes + 2 * (N - 1) * N * chunk_bytes
    row = {"config": "cfg2", "ranks": N, "n_per_rank": 1 << 24, "bound": "REL 0.001", "status": rc,
           "allreduce_us_mean": round(ar_mean, 1), "allreduce_us_best": round(ar_best, 1),
           "allreduce_codec_gbs": round(units / ar_mean / 1e3, 1),
           "allreduce_algbw_gbs": round(4 * (1 << 24) / ar_mean / 1e3, 1),
           "ratio_per_step": per_step, "max_abs_err_vs_fp64_sum": err, "eb_abs": REL * (hi - lo),
           "err_over_eb": round(err / (REL * (hi - lo)), 3)}
    if orc:
        import oracle
        t0 = time.perf_counter()
        oracle.sim_allreduce(send_h, oracle.EB_REL, REL)
        dt = time.perf_counter() - t0
        row["oracle_allreduce_s"] = round(dt, 2)
        row["oracle_codec_gbs"] = round(units / dt / 1e9, 3)
    emit(row)


# --------------------------------------------------------------------------------------------- CUDA arm

def other_configs(z, peak: float, x1, loc1, sm_mhz=None) -> dict:
    """The configurations the step itself does not cover, timed like the rows of --table (10 warm-up + 10 timed graph
    replays per call): cfg1 at the looser and the tighter bound (all three calls), cfg3 (1 GiB gradient-like array,
    compress and decompress) and cfg2 at full size (emulated 8-rank ring Allreduce of 64 MiB per rank).  `frac` =
    algorithmic bytes (input + output of the call, the input twice where a relative bound adds the range pass) / time /
    the measured copy bandwidth."""
    import torch
    from paper_2502_18554_b200 import fields
    out = {}

    def fracs(row):
        nbytes, cbytes = row["bytes"], row["bytes"] / row["ratio"]
        range_bytes = nbytes if str(row.get("bound", "")).startswith("REL") else 0   # a relative bound reads the input once more
        r = {"ratio": row["ratio"], "status": row["status"],
             "compress_us": row["compress_us_mean"],
             "compress_frac": round((range_bytes + nbytes + cbytes) / row["compress_us_mean"] / 1e3 / peak, 3),
             "decompress_us": row["decompress_us_mean"], "decompress_frac": round((nbytes + cbytes) / row["decompress_us_mean"] / 1e3 / peak, 3),
             "compress_gbs": row["compress_gbs"], "decompress_gbs": row["decompress_gbs"]}
        if "fused_us_mean" in row:
            fbytes = nbytes / row["fused_out_ratio"]
            r.update({"fused_us": row["fused_us_mean"], "fused_gbs": row["fused_gbs"],
                      "fused_frac": round((cbytes + nbytes + fbytes) / row["fused_us_mean"] / 1e3 / peak, 3)})
        return r

    big = z.Context(1 << 28, 1)
    for eb in (1e-2, 1e-4):
        out[f"cfg1 REL {eb:g}"] = fracs(_codec_row(z, big, "cfg1", x1, z.EB_REL, eb, False, loc1))
    # the cfg1 field four and sixteen times over (256 MiB, 1 GiB), absolute bound: what the calls reach when their fixed costs
    # (launch ramps, the first round trip, the placement's tail) weigh less
    ebx1 = REL * float(x1.max() - x1.min())
    for reps in (4, 16):
        xr, lr = np.tile(x1, reps), np.tile(loc1, reps)
        out[f"cfg1 x{reps} ({reps * 64} MiB) ABS"] = fracs(_codec_row(z, big, f"cfg1 x{reps}", xr, z.EB_ABS, ebx1, False, lr))
        del xr, lr
    out["cfg3 ABS 1e-05 (1 GiB)"] = fracs(_codec_row(z, big, "cfg3", fields.gradient_like(1 << 28, seed=3), z.EB_ABS, 1e-5, False))
    # the hop with both operands compressed (a variant: the paper's hop adds the rank's own uncompressed chunk).  It moves
    # about 2 bytes per element, so HBM is not what bounds it: `issue_frac` states it against the issue rate instead
    # (thread-instructions per element from an ncu capture of this launch x elements / time / (SMs x 4 schedulers x 32
    # lanes x SM clock)).
    n = x1.size
    sets = 6
    ebx = REL * float(x1.max() - x1.min())
    cap = z.compress_bound(n)
    sz = torch.zeros(1, dtype=torch.int64, device="cuda")
    xa, xb = torch.from_numpy(x1).cuda(), torch.from_numpy(loc1).cuda()
    sa = [torch.empty(cap, dtype=torch.uint8, device="cuda") for _ in range(sets)]
    sb = [torch.empty(cap, dtype=torch.uint8, device="cuda") for _ in range(sets)]
    so = [torch.empty(cap, dtype=torch.uint8, device="cuda") for _ in range(sets)]
    for i in range(sets):
        big.compress(xa, z.EB_ABS, ebx, sa[i], sz)
        ca = int(sz.item())
        big.compress(xb, z.EB_ABS, ebx, sb[i], sz)
        cb = int(sz.item())
    h_us, _ = _timed(lambda i: big.decompress_reduce_compress(sa[i][:ca], n, so[i], sz, local_c=sb[i][:cb]), sets)
    rc = big.check()
    co = int(sz.item())
    props = torch.cuda.get_device_properties(0)
    issue_peak = props.multi_processor_count * 4 * 32 * sm_mhz * 1e6 if sm_mhz else None
    out["cfg1 hop, both operands compressed (ABS)"] = {
        "status": rc, "fused_us": round(h_us, 2), "ratio_in": round(4 * n / ca, 3), "ratio_out": round(4 * n / co, 3),
        "algorithmic_bytes": ca + cb + co, "hbm_frac": round((ca + cb + co) / h_us / 1e3 / peak, 3), "bound": "alu",
        "thread_instructions_per_element": HOP_C2_INSTR_PER_ELEMENT,
        "issue_frac": round(HOP_C2_INSTR_PER_ELEMENT * n / (h_us * 1e-6) / issue_peak, 3) if issue_peak else None}
    del xa, xb, sa, sb, so
    # cfg1 in tiles of 5120 elements, the paper's chunk (encode_rounds_tiled + place_tiled, decode_tiles_tiled)
    out["cfg1 tile 5120 ABS"] = fracs(_tiled_row(z, big, "cfg1, tile of 5120", x1, z.EB_ABS, REL * float(x1.max() - x1.min()), 5120))
    # the cfg1 field as binary64 (128 MiB) through the binary64 entry points (encode_rounds_f64 + place, decode_tiles_f64)
    n = x1.size
    sets = 4
    xd = [torch.from_numpy(x1.astype(np.float64)).cuda() for _ in range(sets)]
    od = [torch.empty(z.compress_bound(n), dtype=torch.uint8, device="cuda") for _ in range(sets)]
    yd = [torch.empty(n, dtype=torch.float64, device="cuda") for _ in range(sets)]
    szd = torch.zeros(1, dtype=torch.int64, device="cuda")
    c_us, _ = _timed(lambda i: big.compress_f64(xd[i], z.EB_REL, REL, od[i], szd), sets)
    rc = big.check()
    cb = int(szd.item())
    d_us, _ = _timed(lambda i: big.decompress_f64(od[i][:cb], yd[i]), sets)
    big.check()
    eb_abs64 = REL * float(x1.max() - x1.min())
    ca_us, _ = _timed(lambda i: big.compress_f64(xd[i], z.EB_ABS, eb_abs64, od[i], szd), sets)
    big.check()
    cba = int(szd.item())
    out["cfg1 as binary64 REL 0.001"] = {
        "ratio": round(8 * n / cb, 3), "status": rc, "compress_us": round(c_us, 2), "decompress_us": round(d_us, 2),
        "compress_gbs": round(8 * n / c_us / 1e3, 1), "decompress_gbs": round(8 * n / d_us / 1e3, 1),
        "compress_frac": round((2 * 8 * n + cb) / c_us / 1e3 / peak, 3),   # the range pass reads the input once more
        "compress_abs_us": round(ca_us, 2), "compress_abs_frac": round((8 * n + cba) / ca_us / 1e3 / peak, 3),
        "decompress_frac": round((8 * n + cb) / d_us / 1e3 / peak, 3),
        "max_abs_err": float((yd[0] - xd[0]).abs().max().item())}
    del xd, od, yd
    big.close()
    torch.cuda.empty_cache()

    N = RANKS
    ctx = z.Context(1 << 27, N)
    send = [torch.from_numpy(a).cuda() for a in fields.rank_fields(N, 1 << 24, base_seed=100)]
    recv = [torch.empty(1 << 24, dtype=torch.float32, device="cuda") for _ in range(N)]
    ar_mean, ar_best = _timed(lambda i: ctx.sim_allreduce(send, recv, z.EB_REL, REL), 1)
    rc = ctx.check()
    chunk_bytes = 4 * (1 << 21)
    units = N * chunk_bytes + 2 * (N - 1) * N * chunk_bytes
    out["cfg2 allreduce 8 x 64 MiB REL 0.001"] = {
        "status": rc, "allreduce_us": round(ar_mean, 1), "allreduce_us_best": round(ar_best, 1),
        "codec_gbs": round(units / ar_mean / 1e3, 1), "algbw_gbs": round(4 * (1 << 24) / ar_mean / 1e3, 1)}
    ctx.close()
    del send, recv
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--min-ms", type=float, default=MIN_TIMED_MS,
                    help="shortest timed region in ms (steps and per-call loops are replayed to get there); 0 for a profiler's launch list")
    ap.add_argument("--no-configs", action="store_true", help="leave the `configs` object (cfg1 at other bounds, cfg2, cfg3) out")
    ap.add_argument("--no-graph", action="store_true", help="time eagerly launched steps instead of CUDA graph replays")
    ap.add_argument("--table", action="store_true",
                    help="time configurations 0-4 one by one (one JSON line per row) instead of the benchmark step")
    ap.add_argument("--rows", default="cfg0,cfg1,cfg2,cfg3,cfg4,collectives",
                    help="with --table: which groups of rows to run (comma-separated)")
    args = ap.parse_args()
    if args.table:
        return config_table(args)
    ref = args.impl == "reference"
    if args.steps is None:
        args.steps = 20 if ref else 1000    # the oracle needs about 0.4 s per step, the GPU under 1 ms
    if args.warmup is None:
        args.warmup = 2 if ref else 10
    if ref:
        return reference_arm(args)
    if args.warmup < 3:
        args.warmup = 3

    import torch
    import torch.distributed as dist
    from paper_2502_18554_b200 import build, zccl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback (use --impl reference for the oracle)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    z = zccl
    ctx = z.Context(N_ELEMS, RANKS)

    # ---- inputs: one batch per rank, copied into ROT rotating sets (distinct memory, > L2 each) by rolling it
    x_h, loc_h = make_fields(rank)
    shift = 4096 * 37
    xs = [torch.from_numpy(np.roll(x_h, k * shift)).to(dev) for k in range(ROT)]
    locs = [torch.from_numpy(np.roll(loc_h, k * shift)).to(dev) for k in range(ROT)]
    cap = z.compress_bound(N_ELEMS)
    cs = [torch.empty(cap, dtype=torch.uint8, device=dev) for _ in range(ROT)]
    c2s = [torch.empty(cap, dtype=torch.uint8, device=dev) for _ in range(ROT)]
    ys = [torch.empty(N_ELEMS, dtype=torch.float32, device=dev) for _ in range(ROT)]
    ars = [torch.empty(N_ELEMS, dtype=torch.float32, device=dev) for _ in range(ROT)]
    ags = [torch.empty(RANKS * RANKS * AG_PER_RANK, dtype=torch.float32, device=dev) for _ in range(ROT)]
    nb1 = torch.zeros(1, dtype=torch.int64, device=dev)
    nb2 = torch.zeros(1, dtype=torch.int64, device=dev)
    per = N_ELEMS // RANKS
    stream = torch.cuda.current_stream()

    names = ["compress", "decompress", "fused", "allreduce", "allgather"]

    def step(i: int, evs=None):
        k = i % ROT
        x, loc, c, c2, y, ar, ag = xs[k], locs[k], cs[k], c2s[k], ys[k], ars[k], ags[k]
        if evs is not None:
            evs[0].record(stream)
        ctx.compress(x, z.EB_REL, REL, c, nb1)
        if evs is not None:
            evs[1].record(stream)
        ctx.decompress(c, y)
        if evs is not None:
            evs[2].record(stream)
        ctx.decompress_reduce_compress(c, N_ELEMS, c2, nb2, local=loc)
        if evs is not None:
            evs[3].record(stream)
        ctx.sim_allreduce([x[r * per:(r + 1) * per] for r in range(RANKS)],
                          [ar[r * per:(r + 1) * per] for r in range(RANKS)], z.EB_REL, REL)
        if evs is not None:
            evs[4].record(stream)
        ctx.sim_allgather([x[r * AG_PER_RANK:(r + 1) * AG_PER_RANK] for r in range(RANKS)],
                          [ag[r * RANKS * AG_PER_RANK:(r + 1) * RANKS * AG_PER_RANK] for r in range(RANKS)],
                          z.EB_REL, REL)
        if evs is not None:
            evs[5].record(stream)

    def fence():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    ctx.check()
    ratio1 = 4 * N_ELEMS / int(nb1.item())
    ratio2 = 4 * N_ELEMS / int(nb2.item())

    # ---- timed region: the step replayed from CUDA graphs (one per rotating buffer set), which removes the launch gaps
    # between its 23 short kernels; the work and the results are those of the eager step (tests/test_gpu_parity.py
    # replays a captured step against the oracle).  If capture is not possible the eager step is timed instead.
    graphs = None
    launches_per_step = None
    if not args.no_graph:
        try:
            side = torch.cuda.Stream()
            side.wait_stream(stream)
            graphs = []
            with torch.cuda.stream(side):
                for k in range(ROT):
                    step(k)
                torch.cuda.synchronize()
                for k in range(ROT):
                    l0 = z.launch_count()
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=side):
                        step(k)
                    launches_per_step = z.launch_count() - l0
                    graphs.append(g)
                for g in graphs:
                    g.replay()
            torch.cuda.synchronize()
            ctx.check()
        except Exception as exc:   # noqa: BLE001 - any failure to capture falls back to the eager step
            print(f"bench: CUDA graph capture failed ({exc!r}); timing the eager step", file=sys.stderr)
            graphs = None

    # Every step is run `replays` times in a row, so that the timed region lasts half a second or more whatever
    # --steps says (the clock sampler then sees it, and the figure does not depend on the run's length); ms_per_step
    # stays the time of ONE pass.  All ranks use the same count.
    replays = 1
    if graphs is not None:
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        p0.record(stream)
        for k in range(ROT):
            graphs[k].replay()
        p1.record(stream)
        p1.synchronize()
        est_ms = max_over_ranks(p0.elapsed_time(p1), dev) / ROT
        replays = max(1, int(-(-args.min_ms // (est_ms * args.steps))))
    sampler = ClockSampler(local_rank)
    fence()
    sampler.start()
    time.sleep(0.25)            # the sampler's first line takes this long to come
    launches0 = z.launch_count()
    t_begin = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_begin.record(stream)
    for i in range(args.steps):
        if graphs is not None:
            for _ in range(replays):
                graphs[(args.warmup + i) % ROT].replay()
        else:
            step(args.warmup + i)
    t_end.record(stream)
    fence()
    launches = (launches_per_step * args.steps * replays) if graphs is not None else (z.launch_count() - launches0)
    clocks = sampler.stop()
    ctx.check()
    ms_total = max_over_ranks(t_begin.elapsed_time(t_end), dev)
    ms_step = ms_total / (args.steps * replays)
    units = step_units_bytes()
    total_bytes = sum(units.values())
    value = whole_job_gbs(total_bytes, world, ms_step)

    # ---- the same steps once more, launched eagerly with an event after every operation: time per operation
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(6)] for _ in range(args.steps)]
    e_begin = torch.cuda.Event(enable_timing=True)
    e_end = torch.cuda.Event(enable_timing=True)
    fence()
    e_begin.record(stream)
    for i in range(args.steps):
        step(args.warmup + i, evs[i])
    e_end.record(stream)
    fence()
    ctx.check()
    ms_step_eager = max_over_ranks(e_begin.elapsed_time(e_end), dev) / args.steps
    op_ms = {nm: statistics.mean(evs[i][j].elapsed_time(evs[i][j + 1]) for i in range(args.steps))
             for j, nm in enumerate(names)}

    # ---- roofline of the codec's three calls, each timed by itself: back-to-back calls replayed from a CUDA graph over
    # the rotating buffer sets, at least 200 of them and at least 0.4 s, inside one pair of events, with the SM clock
    # sampled meanwhile.  compress is timed with the pre-resolved absolute bound (a relative bound adds the range pass):
    # two launches (rounds into slots, then placement); decompress is one launch; the fused hop two (hop, placement).
    peaks = {}
    pk = ROOT / "MEASURED_PEAKS.json"
    peak_src = "fallback"
    peak = 6650.0
    if pk.exists():
        try:
            peaks = json.loads(pk.read_text())
            peak = float(peaks["hbm_gbs"]); peak_src = "measured"
        except Exception:
            pass
    eb_abs = float(np.float32(REL) * (np.float32(x_h.max()) - np.float32(x_h.min())))
    for k in range(ROT):                       # the streams the decoder and the hop read
        ctx.compress(xs[k], z.EB_REL, REL, cs[k], nb1)
    torch.cuda.synchronize()
    kmin_ms, kmin_n = (400.0, 200) if args.min_ms > 0 else (0.0, 2 * ROT)
    enc_us, enc_calls, enc_mhz = _timed_long(lambda k: ctx.compress(xs[k], z.EB_ABS, eb_abs, c2s[k], nb2), ROT, local_rank, kmin_ms, kmin_n)
    dec_us, dec_calls, dec_mhz = _timed_long(lambda k: ctx.decompress(cs[k], ys[k]), ROT, local_rank, kmin_ms, kmin_n)
    hop_us, hop_calls, hop_mhz = _timed_long(
        lambda k: ctx.decompress_reduce_compress(cs[k], N_ELEMS, c2s[k], nb2, local=locs[k]), ROT, local_rank, kmin_ms, kmin_n)
    ctx.check()
    in_b = 4 * N_ELEMS
    c1_b = in_b / ratio1
    c2_b = in_b / ratio2
    kern = {
        "encode(compress, ABS bound): encode_rounds + place": {"ms": enc_us * 1e-3, "bytes": in_b + c1_b, "calls": enc_calls, "sm_mhz": enc_mhz},
        "decode(decompress): decode_tiles": {"ms": dec_us * 1e-3, "bytes": c1_b + in_b, "calls": dec_calls, "sm_mhz": dec_mhz},
        "encode_fused(decompress-add-recompress): hop_tiles + place": {"ms": hop_us * 1e-3, "bytes": c1_b + in_b + c2_b, "calls": hop_calls,
                                                                     "sm_mhz": hop_mhz},
    }
    for v in kern.values():
        v["achieved_gbs"] = v["bytes"] / (v["ms"] * 1e-3) / 1e9
        v["frac"] = v["achieved_gbs"] / peak
        v["frac_of_nominal_8000"] = v["achieved_gbs"] / 8000.0   # the nominal HBM3e figure, for context
        v["uncompressed_gbs"] = in_b / (v["ms"] * 1e-3) / 1e9
        v["us_x_mhz"] = v["ms"] * 1e3 * v["sm_mhz"] if v["sm_mhz"] else None   # clock-independent cost: cycles per call
    # the fused kernel also runs the 56 chunk hops of the allreduce: it carries the largest share of the step
    dom = "encode_fused(decompress-add-recompress): hop_tiles + place"
    roofline = {"bound": "hbm", "kernel": dom, "achieved": kern[dom]["achieved_gbs"], "peak": peak, "unit": "GB/s",
                "frac": kern[dom]["frac"], "frac_of_nominal_8000": kern[dom]["frac_of_nominal_8000"], "traffic": None,
                "peak_source": f"of {peak_src}",
                "algorithmic_bytes_per_launch": kern[dom]["bytes"]}
    roofline["traffic"] = DRAM_TRAFFIC_FUSED_64MIB

    # ---- quality of the reconstruction (Section 4.1: NRMSE, PSNR, bit rate), and the metrics kernel's own roofline
    # (it reads both arrays once: 8 bytes per element, nothing else)
    qout = torch.zeros(6, dtype=torch.float64, device=dev)
    for k in range(ROT):
        ctx.compress(xs[k], z.EB_REL, REL, cs[k], nb1)
        ctx.decompress(cs[k], ys[k])
    q_us, q_calls, q_mhz = _timed_long(lambda k: ctx.quality(xs[k], ys[k], qout), ROT, local_rank, kmin_ms, kmin_n)
    ctx.quality(xs[0], ys[0], qout)   # the batch the ratios are quoted on
    torch.cuda.synchronize()
    qv = qout.cpu().numpy()
    hist = torch.zeros(33, dtype=torch.int64, device=dev)
    ctx.stream_stats(cs[0], hist)     # the stream of the batch the ratios are quoted on (length from its header)
    ctx.check()
    hh = hist.cpu().numpy().astype(np.float64)
    quality = {"max_abs_err": float(qv[0]), "nrmse": float(qv[2]), "psnr_db": float(qv[3]), "bit_rate": 32.0 / ratio1,
               "eb_abs": eb_abs, "constant_block_pct": 100.0 * hh[0] / max(hh[32], 1.0),
               "mean_code_length": float((hh[:32] * np.arange(32)).sum() / max(hh[32], 1.0))}
    kern["quality(metrics)"] = {"ms": q_us * 1e-3, "bytes": 2.0 * in_b, "calls": q_calls, "sm_mhz": q_mhz,
                                "us_x_mhz": q_us * q_mhz if q_mhz else None}
    kq = kern["quality(metrics)"]
    kq["achieved_gbs"] = kq["bytes"] / (kq["ms"] * 1e-3) / 1e9
    kq["frac"] = kq["achieved_gbs"] / peak
    kq["frac_of_nominal_8000"] = kq["achieved_gbs"] / 8000.0
    kq["uncompressed_gbs"] = in_b / (kq["ms"] * 1e-3) / 1e9

    # ---- end to end through the host-buffer entry points (pinned host memory; copies inside the timed region)
    xh = torch.from_numpy(x_h).pin_memory()
    oh = torch.empty(cap, dtype=torch.uint8).pin_memory()
    yh = torch.empty(N_ELEMS, dtype=torch.float32).pin_memory()
    e2e_steps = max(3, min(args.steps, 10))
    for _ in range(2):
        nb = ctx.compress_host(xh, z.EB_REL, REL, oh)
        ctx.decompress_host(oh, nb, yh)
    fence()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        nb = ctx.compress_host(xh, z.EB_REL, REL, oh)
        ctx.decompress_host(oh, nb, yh)
    e1.record(stream)
    fence()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), dev) / e2e_steps
    e2e = {"value": whole_job_gbs(2 * in_b, world, e2e_ms), "unit": "GB/s",
           "what": "zccl_compress_host + zccl_decompress_host of the 64 MiB batch (uncompressed bytes per op / time)",
           "ms_per_step": e2e_ms, "h2d_bytes_per_step": in_b + nb, "d2h_bytes_per_step": nb + 8 + in_b}

    # The same pairs as two independent pipelines (a context and a stream each, taking turns): one pipeline's upload
    # runs while the other's download does, which is what a PCIe link's two directions allow; a single call chain can
    # only use one direction at a time.
    ctx_b = z.Context(N_ELEMS, 0)
    pipes = [(ctx, torch.cuda.Stream(), oh, yh),
             (ctx_b, torch.cuda.Stream(), torch.empty(cap, dtype=torch.uint8).pin_memory(), torch.empty(N_ELEMS, dtype=torch.float32).pin_memory())]
    for c, s_, o_, y_ in pipes:
        c.decompress_host(o_, c.compress_host(xh, z.EB_REL, REL, o_, stream=s_), y_, stream=s_)
    fence()
    p0 = torch.cuda.Event(enable_timing=True)
    p0.record(pipes[0][1])
    for _ in range(e2e_steps):
        for c, s_, o_, y_ in pipes:
            c.decompress_host(o_, c.compress_host(xh, z.EB_REL, REL, o_, stream=s_), y_, stream=s_)
    ends = []
    for c, s_, o_, y_ in pipes:
        e_ = torch.cuda.Event(enable_timing=True)
        e_.record(s_)
        ends.append(e_)
    fence()
    ctx.check()
    ctx_b.check()
    two_ms = max_over_ranks(max(p0.elapsed_time(e_) for e_ in ends), dev) / (2 * e2e_steps)
    e2e["two_pipelines"] = {"value": whole_job_gbs(2 * in_b, world, two_ms), "unit": "GB/s", "ms_per_step": two_ms,
                            "what": "the same pairs issued in turn on two contexts and two streams"}
    ctx_b.close()

    # ---- the other configurations of the workload list, a few graph replays each (single-GPU runs only)
    configs = None
    if rank == 0 and world == 1 and not args.no_configs:
        ctx.close()
        ctx = None
        del xs, locs, cs, c2s, ys, ars, ags
        torch.cuda.empty_cache()
        configs = other_configs(z, peak, x_h, loc_h, clocks.get("sm_mhz") if clocks else None)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        oracle.build()
        sample = N_ELEMS // 4
        reps = 4
        gbs, ms = run_oracle(x_h, loc_h, reps, 1, sample)
        cpu = {"value": gbs, "unit": "GB/s", "cores": 1, "kind": "oracle", "host_cores": os.cpu_count(),
               "sample": f"{reps} steps on the first {sample} of {N_ELEMS} elements of the batch (one quarter), "
                         f"{ms * reps / 1e3:.1f} s of CPU work"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": WORKLOAD, "l2": f"inputs and outputs rotate over {ROT} buffer sets, each above L2",
                       "rel_bound": REL, "ratio_compress": ratio1, "ratio_fused_out": ratio2,
                       "parallelism": f"{world} independent replicas" if world > 1 else "single GPU",
                       "launch": "CUDA graph replay, one graph per buffer set" if graphs is not None else "eager",
                       "timed_region_ms": ms_total},
            "replays_per_step": replays,
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
            "roofline": roofline, "cpu_baseline": cpu,
            "ms_per_step_eager": ms_step_eager, "ops_ms": op_ms, "ops_uncompressed_gbs": {nm: units[nm] / (op_ms[nm] * 1e-3) / 1e9 for nm in names},
            "kernels": kern, "quality": quality, "configs": configs,
        }
        print(json.dumps(line))
    if ctx is not None:
        ctx.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
