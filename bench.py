#!/usr/bin/env python
"""Benchmark of the DaSGD hot path (local step + snapshot + worker-axis mean + delayed merge).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload resnet50|...]

One "step" is one pass of the whole path over one batch of synthetic gradients: a local step of
all K replicas, the merge that lands on that step, the snapshot and the side-stream mean.
Workload "resnet50": K=8 replicas of a P=25.6M float32 vector, momentum 0.9, weight decay 1e-4,
lr 0.1, tau=1, d=1, xi=0.25.  Prints ONE JSON line (rank 0).

The timed loop of K steps is repeated (--repeats, default 5) and the median is reported, with the
minimum and maximum beside it.  With --gpus N > 1 and no launcher in the environment the script starts
its N ranks itself (torch.distributed.run on 127.0.0.1).

--impl reference times the plain CPU checker under oracle/ on the host cores, on a bounded slice of
the same workload (the path is independent across the parameter index, so a slice is exact).
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2006_00441_b200 import inputs  # noqa: E402

WORKLOADS = {
    # name: K, P, momentum, weight_decay, lr, tau, d, xi, grad std, w0 std
    "resnet50": dict(K=8, P=25_600_000, momentum=0.9, weight_decay=1e-4, lr=0.1, tau=1, d=1, xi=0.25,
                     g_std=1e-3 ** 0.5, w_std=0.02),
    "small": dict(K=4, P=1024, momentum=0.0, weight_decay=0.0, lr=0.01, tau=4, d=1, xi=0.25,
                  g_std=1.0, w_std=0.0),
    # BERT-large-sized: bfloat16 gradients and weight copy, float32 master weights / momentum
    "bert_large": dict(K=4, P=335_000_000, momentum=0.9, weight_decay=0.0, lr=1e-3, tau=2, d=1, xi=0.25,
                       g_std=1e-2, w_std=0.02, bf16=True, ring=2),
}
METRIC = "replica-param updates/s"
UNIT = "updates/s"
CHUNK_BYTES = 18 << 20   # target size of one column range of the weight array in the column-range pipeline
HOST_US_PER_RANGE = 20.0  # host time to enqueue one range (four CUDA calls, about 14 us measured) with some margin:
                          # more ranges than the iteration has time for would make the host the bottleneck
MIN_RANGE_COLS = 409_600  # narrower ranges leave the mean kernel too few columns to fill the GPU (K >= 16)


def step_bytes(wl):
    """Algorithmic HBM bytes per replica-parameter of one plain local-step launch."""
    if wl.get("bf16"):
        return (2 + 4 + 4 + 4 + 4 + 2) if wl["momentum"] else (2 + 4 + 4 + 2)
    return 20 if wl["momentum"] else 12   # read w, (m,) g; write w (, m)


def auto_chunks(K, P, bytes_per_update=25.0):
    """Column ranges of the pipeline: ranges of about CHUNK_BYTES of the [K][P] weight array (small enough
    that the mean of a range finds much of it still in L2), but no more than the host can enqueue in the time
    the GPU needs for one iteration (estimated at the measured copy bandwidth)."""
    by_size = round(K * P * 4 / CHUNK_BYTES)
    iteration_us = K * P * bytes_per_update / (measured_peak_gbs()[0] * 1e9) * 1e6
    return int(max(2, min(1024, by_size, iteration_us / HOST_US_PER_RANGE, P / MIN_RANGE_COLS)))


def schedule_of(wl, args):
    """How bench.py runs dasgd_step for this workload: {'merge': 'chunked'|'fused'|'separate', 'n_chunks', 'lanes'}."""
    if args.no_fuse:
        return {"merge": "separate", "n_chunks": 0, "lanes": 0, "copy_snapshot": True}
    if wl["d"] >= 1 and args.chunks != 1 and wl["P"] >= 2 * 4096:
        n = args.chunks if args.chunks > 0 else auto_chunks(wl["K"], wl["P"])
        return {"merge": "chunked", "n_chunks": n, "lanes": 1 if args.lanes else 0, "graph": 1 if args.graph else 0,
                "side_streams": 2 if args.sides == 2 and wl["K"] >= 4 else 1}   # K = 2: one side stream measured 2 % faster
    if wl["d"] >= 2:
        return {"merge": "fused", "n_chunks": 0, "lanes": 0}
    return {"merge": "separate", "n_chunks": 0, "lanes": 0}


def path_bytes_per_update(wl, sched):
    """Algorithmic HBM bytes per replica-parameter update of the whole path as scheduled: tau local
    steps, the snapshot (0 B with rotating arrays, 8 B as a copy), the mean (4 + 4/K B), and the merge
    (4/K B when folded into a step kernel, else a pass of its own: 8 + 4/K B, + 2 B for the bfloat16 copy)."""
    K, tau = wl["K"], wl["tau"]
    per_cycle = step_bytes(wl) * tau + (4.0 + 4.0 / K)
    if sched.get("copy_snapshot"):
        per_cycle += 8.0
    if sched["merge"] in ("chunked", "fused"):
        per_cycle += 4.0 / K
    else:
        per_cycle += 8.0 + 4.0 / K + (2.0 if wl.get("bf16") else 0.0)
    return per_cycle / tau


# DRAM traffic of the dominant kernel from an ncu capture (profiles/): k_local_step_vec<f32, momentum, xi-merge>
# on one column range of the pipeline.  Reads grow with the updates of a launch; the stores that are still
# dirty in L2 when the kernel ends are a constant, not a share.  Valid only while the kernel source is the
# one that was profiled.
NCU_TRAFFIC = {"kernels_sha256_prefix": "ae8627e365d3f6a1", "updates": 5_275_648, "read_bytes": 65.965e6, "write_bytes": 2.40e6,
               "applies_to": "float32 + momentum, merge folded in"}


def profiled_traffic(wl, sched, updates_per_launch):
    """DRAM bytes of one launch of the dominant kernel derived from the last ncu capture, or None when the
    kernels have changed since or the workload is not the profiled variant."""
    import hashlib
    if not NCU_TRAFFIC["kernels_sha256_prefix"] or wl.get("bf16") or not wl["momentum"] or sched["merge"] != "chunked":
        return None
    try:
        src = os.path.join(ROOT, "paper_2006_00441_b200", "csrc", "dasgd_kernels.cuh")
        if hashlib.sha256(open(src, "rb").read()).hexdigest()[:16] != NCU_TRAFFIC["kernels_sha256_prefix"]:
            return None
    except OSError:
        return None
    n0 = NCU_TRAFFIC["updates"]
    residue = max(0.0, 8.0 * n0 - NCU_TRAFFIC["write_bytes"])          # dirty lines left in L2: constant
    reads = NCU_TRAFFIC["read_bytes"] * updates_per_launch / n0         # proportional
    writes = max(0.0, 8.0 * updates_per_launch - residue)
    return reads + writes


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# ------------------------------------------------------------------ clocks

class ClockSampler:
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.proc, self.path = None, None
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            ident = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", ident, f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self, window=None):
        """Median SM clock and the throttle reasons seen.  `window` = (t0, t1) in time.time() seconds: only the
        samples taken inside it count (the sampler is started well before, because nvidia-smi needs a moment to
        come up); if none falls inside, all samples do, and the summary says so."""
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        import datetime
        rows = []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 8:
                    continue
                try:
                    ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    rows.append((ts, float(f[1]), float(f[2]), [nm for nm, v in zip(names, f[4:8]) if v.lower().startswith("active")]))
                except ValueError:
                    continue
            os.unlink(self.path)
        except Exception:
            pass
        inside = [r for r in rows if window and window[0] <= r[0] <= window[1]]
        used = inside or rows
        if used:
            out["sm_mhz"] = statistics.median(r[1] for r in used)
            out["sm_max_mhz"] = max(r[2] for r in used)
        out["reasons"] = sorted({nm for r in used for nm in r[3]})
        out["samples"] = len(used)
        out["window"] = "timed region" if inside else "whole measurement (no sample fell inside the timed region)"
        return out


# ------------------------------------------------------------------ CPU oracle legs

def oracle_throughput(wl, seconds_budget: float, steps: int | None = None, warmup: int = 0, omp: bool = True):
    """Times the CPU checker on the first P_s parameters of every replica.  Returns a dict."""
    import numpy as np

    import oracle

    K = wl["K"]
    probe = oracle.OracleDaSGD(K, 1, 1, 1, 0.5, omp=omp)
    cores = probe.threads
    probe.close()
    # calibrate on a slice too large for the CPU caches, so the rate is the DRAM-bound one
    Pc = min(wl["P"], 2_000_000)
    odt = 1 if wl.get("bf16") else 0

    def host_grad(t, idx):
        g = inputs.grad_block(0, t, K, wl["P"], wl["g_std"], p_index=idx,
                              dtype=torch.bfloat16 if odt else torch.float32)
        return g.view(torch.int16).numpy().view(np.uint16) if odt else g.numpy()

    o = oracle.OracleDaSGD(K, Pc, wl["tau"], wl["d"], wl["xi"], wl["momentum"], wl["weight_decay"], dtype=odt, omp=omp)
    o.set_state(inputs.shared_start(0, wl["P"], wl["w_std"], p_index=range(Pc)).numpy())
    g = host_grad(0, range(Pc))
    for _ in range(2):
        o.step(g, wl["lr"])
    t0 = time.perf_counter()
    n_cal = 5
    for _ in range(n_cal):
        o.step(g, wl["lr"])
    rate = K * Pc * n_cal / (time.perf_counter() - t0)  # updates/s, rough
    if steps is None:       # cpu_baseline leg: fixed slice, as many steps as fit the budget
        Ps = Pc
        steps = max(3, min(200, int(seconds_budget * rate / (K * Ps))))
        ring = [g, host_grad(1, range(Ps))]
    else:                   # reference arm: the caller fixes the steps, the slice is sized to the budget
        o.close()
        Ps = int(min(wl["P"], 4_000_000, max(1024, seconds_budget * rate / (K * (steps + warmup)))))
        idx = range(Ps)
        o = oracle.OracleDaSGD(K, Ps, wl["tau"], wl["d"], wl["xi"], wl["momentum"], wl["weight_decay"], dtype=odt, omp=omp)
        o.set_state(inputs.shared_start(0, wl["P"], wl["w_std"], p_index=idx).numpy())
        ring = [host_grad(t, idx) for t in range(2)]
    for t in range(warmup):
        o.step(ring[t % 2], wl["lr"])
    t0 = time.perf_counter()
    for t in range(steps):
        o.step(ring[t % 2], wl["lr"])
    dt = time.perf_counter() - t0
    assert np.isfinite(o.w).all()
    o.close()
    build = f"OpenMP build of the checker, {cores} threads" if omp else "plain single-thread build of the checker"
    return {"value": K * Ps * steps / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {Ps} of {wl['P']} parameters of all {K} replicas, {steps} steps ({build})",
            "seconds": dt, "steps": steps, "P_sample": Ps}


def cpu_baseline(wl):
    """The checker as it stands on the host cores: all cores (OpenMP build) and one thread (plain build)."""
    par = oracle_throughput(wl, seconds_budget=12.0, omp=True)
    one = oracle_throughput(wl, seconds_budget=6.0, omp=False)
    out = {k: par[k] for k in ("value", "unit", "cores", "kind", "sample")}
    out["single_thread"] = {k: one[k] for k in ("value", "unit", "cores", "sample")}
    return out


def run_reference(args, wl, name):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    r = oracle_throughput(wl, seconds_budget=60.0, steps=args.steps, warmup=args.warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * r["seconds"] / r["steps"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 gradients, f32 state" if wl.get("bf16") else "f32", "data": "synthetic",
        "config": workload_config(wl, name, None),
        "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")},
        "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(wl, name, sched, shard="replicas", world=1):
    cfg = {"workload": f"{name}: K={wl['K']} replicas x P={wl['P']} {'bf16 gradients + f32 master' if wl.get('bf16') else 'float32'}, momentum {wl['momentum']}, "
                       f"weight decay {wl['weight_decay']}, lr {wl['lr']}, tau={wl['tau']}, d={wl['d']}, xi={wl['xi']}",
           "K": wl["K"], "P": wl["P"], "tau": wl["tau"], "d": wl["d"], "xi": wl["xi"],
           "l2_policy": "inputs larger than L2 (every step streams all K*P-sized arrays; gradients come from a ring of buffers)",
           "parallelism": "independent replicas of the workload per GPU (no collective on this path)"}
    if shard == "workers":
        cfg["parallelism"] = (f"worker axis sharded: {wl['K']} of {wl['K'] * world} workers per GPU; one ncclAllReduce of the "
                              "partial sums (P float32) per snapshot on the side stream")
        cfg["K_total"] = wl["K"] * world
    if sched is not None:
        cfg["schedule"] = sched
    return cfg


# ------------------------------------------------------------------ our arm

def whole_job(ms_local: float, units_per_rank: float, dist=None, device="cpu"):
    """Whole-job figures from one rank's device time: the job takes as long as its slowest rank
    (MAX over ranks) and processes the units of all ranks.  Returns (ms, units/s)."""
    world = 1
    ms = float(ms_local)
    if dist is not None and dist.is_initialized():
        world = dist.get_world_size()
        tms = torch.tensor([ms], dtype=torch.float64, device=device)
        dist.all_reduce(tms, op=dist.ReduceOp.MAX)
        ms = float(tms.item())
    return ms, world * units_per_rank / (ms * 1e-3)


class Bench:
    """One rank's harness: builds contexts for a workload and times loops of steps on them."""

    def __init__(self, args):
        from paper_2006_00441_b200 import binding as B
        self.B, self.args = B, args
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the path has no CPU implementation")
        torch.cuda.set_device(self.local_rank)
        self.dist = None
        if self.world > 1 or args.force_dist:
            import torch.distributed as dist
            if "RANK" not in os.environ:     # a single rank started without a launcher
                os.environ.update(RANK="0", WORLD_SIZE="1", LOCAL_RANK="0", MASTER_ADDR="127.0.0.1",
                                  MASTER_PORT=str(_free_port()))
            dist.init_process_group("nccl", device_id=torch.device("cuda", self.local_rank))
            self.dist = dist
        # --shard workers: the K workers of every rank are shards of one K*world-worker job; the partial sums
        # are exchanged by the library's own NCCL communicator (rank 0 makes the id, torch broadcasts it)
        self.comm = None
        if args.shard == "workers":
            uid = torch.zeros(128, dtype=torch.uint8)
            if self.rank == 0:
                uid = torch.frombuffer(bytearray(B.dasgd_nccl_unique_id()), dtype=torch.uint8).clone()
            if self.dist is not None:
                dev = uid.cuda()
                self.dist.broadcast(dev, 0)
                uid = dev.cpu()
            self.comm = B.dasgd_nccl_comm_init(bytes(uid.numpy().tobytes()), self.world, self.rank, self.local_rank)

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        torch.cuda.synchronize()

    def flags(self, sched, timing=False):
        B = self.B
        if sched["merge"] == "separate" and sched.get("copy_snapshot"):
            f = 0
        else:
            f = B.DASGD_FLAG_ROTATE_SNAPSHOT | B.DASGD_FLAG_FUSE_MERGE
        if sched.get("lanes"):
            f |= B.DASGD_FLAG_TWO_LANES
        if sched.get("graph"):
            f |= B.DASGD_FLAG_GRAPH
        if sched.get("side_streams") == 2:
            f |= B.DASGD_FLAG_TWO_SIDE_STREAMS
        return f | (B.DASGD_FLAG_TIMING if timing else 0)

    def make(self, wl, sched, timing=False, host_staging=False, flags=None, snapshot_arrays=True):
        B = self.B
        e = B.DaSGD(wl["K"], wl["P"], wl["tau"], wl["d"], wl["xi"], wl["momentum"], wl["weight_decay"],
                    flags=self.flags(sched, timing) if flags is None else flags,
                    dtype=B.DASGD_BF16_MASTER_F32 if wl.get("bf16") else B.DASGD_F32,
                    n_chunks=sched["n_chunks"] if flags is None else 0, device=self.local_rank,
                    host_staging=host_staging, order_after_current=False, snapshot_arrays=snapshot_arrays)
        if self.comm is not None and not (e.cfg.flags & B.DASGD_FLAG_INLINE_MEAN):
            e.set_shard(wl["K"] * self.world, nccl_comm=self.comm)
        # independent replicas: every rank its own start; shards of one job: the common start of all workers
        seed = 1000 if self.comm is not None else 1000 + self.rank
        e.set_state(inputs.shared_start(seed, wl["P"], wl["w_std"], device="cuda"))
        return e

    def timed(self, e, steps, step_fn, t0=0):
        """Device time of `steps` calls of step_fn, bracketed by barrier + synchronize; MAX over ranks."""
        e.sync()
        self.barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0 = e.launches
        with torch.cuda.stream(e.main):
            ev0.record()
        for t in range(steps):
            step_fn(e, t0 + t)
        e.main.wait_stream(e.side)        # the last mean belongs to the timed work
        with torch.cuda.stream(e.main):
            ev1.record()
        e.sync()
        self.barrier()
        ms, _ = whole_job(ev0.elapsed_time(ev1), 0.0, self.dist, "cuda")
        return ms, e.launches - l0

    def repeated(self, e, steps, warmup, repeats, step_fn):
        """Warm-up, then `repeats` timed loops of exactly `steps` steps.  Returns per-step ms (median, min, max)."""
        for t in range(warmup):
            step_fn(e, t)
        per, launches = [], 0
        for r in range(repeats):
            ms, launches = self.timed(e, steps, step_fn, warmup + r * steps)
            per.append(ms / steps)
        return {"ms_per_step": statistics.median(per), "min": min(per), "max": max(per), "repeats": repeats,
                "launches": launches}


def measure_workload(bench, wl, sched, steps, warmup, repeats, ring, lr, with_alone=True):
    """Headline loop + instrumented pass (+ kernels alone) of one workload; returns a dict of figures."""
    K, P = wl["K"], wl["P"]
    RING = len(ring)

    def dev_step(e, t):
        e.step(ring[t % RING], lr)

    out = {}
    eng = bench.make(wl, sched)
    t_begin = time.time()
    out["headline"] = bench.repeated(eng, steps, warmup, repeats, dev_step)
    out["headline_window"] = (t_begin, time.time())     # host clock, for the clock sampler: warm-up + the timed loops
    eng.close()
    del eng

    # ---- instrumented pass: per-kernel device time and the stalls of the averaging
    eng = bench.make(wl, sched, timing=True)
    for t in range(warmup):
        dev_step(eng, t)
    eng.reset_timing()
    n_inst = min(steps, 100)
    for t in range(n_inst):
        dev_step(eng, warmup + t)
    kt = eng.kernel_timing()
    eng.close()
    del eng
    out["kernels_ms_per_launch"] = {k: (v[1] / v[0] if v[0] else None) for k, v in kt.items()}
    out["kernels_ms_per_step"] = {k: v[1] / n_inst for k, v in kt.items()}
    out["kernel_launches_per_step"] = {k: v[0] / n_inst for k, v in kt.items()}
    out["instrumented_steps"] = n_inst
    if kt["mean"][0] and kt["mean"][1] > 0:
        out["hidden"] = max(0.0, 1.0 - kt["stall"][1] / kt["mean"][1])
        out["stall_ms_per_step"] = kt["stall"][1] / n_inst
    else:
        out["hidden"] = None
    if with_alone:
        # the same kernels with nothing else on the GPU (no side-stream mean beside them)
        plain = dict(sched, merge="separate", n_chunks=0, lanes=0)
        eng = bench.make(wl, plain, timing=True)
        for t in range(3):
            eng.local_step(ring[t % RING], lr)
        eng.reset_timing()
        for t in range(20):
            eng.local_step(ring[t % RING], lr)
        eng.sync()
        for t in range(10):
            eng.snapshot(); eng.average_async(); eng.sync(); eng.merge(); eng.sync()
        kt_alone = eng.kernel_timing()
        eng.close()
        del eng
        peak, _ = measured_peak_gbs()
        alone = {}
        bf16 = bool(wl.get("bf16"))
        for kname, nbytes in (("local_step", K * P * step_bytes(wl)), ("mean", K * P * 4 + P * 4),
                              ("merge", K * P * (10 if bf16 else 8) + P * 4)):
            n_k, ms_k = kt_alone[kname]
            if n_k:
                gbs = nbytes / 1e9 / (ms_k / n_k * 1e-3)
                alone[kname] = {"ms": ms_k / n_k, "GB/s": gbs, "frac": gbs / peak}
        out["alone"] = alone
    return out


def calibrate_chunks(bench, wl, sched, ring, lr):
    """The number of column ranges is a trade between L2 residency (more, smaller ranges) and the host's
    enqueue rate (four CUDA calls per range; a slower host needs fewer, longer ranges).  The formula in
    auto_chunks assumes a host like the one it was tuned on, so a short trial decides: 40 steps at each of a few
    counts around the formula's value, the fastest wins.  Returns the schedule with the chosen count."""
    base = sched["n_chunks"]
    cands = sorted({max(2, int(round(base * f))) for f in (0.6, 0.8, 1.0, 1.25)})
    RING = len(ring)
    trials = {}
    for c in cands:
        trial = dict(sched, n_chunks=c)
        eng = bench.make(wl, trial)
        r = bench.repeated(eng, 40, 5, 1, lambda e, t: e.step(ring[t % RING], lr))
        trials[c] = r["ms_per_step"]
        eng.close()
        del eng
    best = min(trials, key=trials.get)
    return dict(sched, n_chunks=best, calibration_ms_per_step={str(k): round(v, 5) for k, v in trials.items()})


def hidden_cost(wl, sched, ms_per_step, alone):
    """1 - (cycle time - cycle time of the main-stream kernels alone) / mean kernel alone."""
    if not all(k in alone for k in ("local_step", "mean", "merge")):
        return None
    tau, K = wl["tau"], wl["K"]
    main_alone = tau * alone["local_step"]["ms"]
    if sched["merge"] == "separate":
        main_alone += alone["merge"]["ms"]
    else:   # folded in: the step kernel that merges also reads the mean once per row
        main_alone += alone["local_step"]["ms"] * (4.0 / K) / step_bytes(wl)
    return 1.0 - (ms_per_step * tau - main_alone) / alone["mean"]["ms"]


def run_ours(args, wl, name, bench=None, compact=False):
    bench = bench or Bench(args)
    B, rank, world = bench.B, bench.rank, bench.world
    K, P, lr = wl["K"], wl["P"], wl["lr"]
    bf16 = bool(wl.get("bf16"))
    gdt = torch.bfloat16 if bf16 else torch.float32
    RING = wl.get("ring", 4)
    sched = schedule_of(wl, args)
    sampler = ClockSampler(bench.local_rank) if rank == 0 and not compact else None   # started early: it takes a moment to come up
    seed = 1000 + rank  # every rank runs its own replica of the workload
    ring = [inputs.grad_block(seed, t, K, P, wl["g_std"], device="cuda", dtype=gdt) for t in range(RING)]
    torch.cuda.synchronize()

    def dev_step(e, t):
        e.step(ring[t % RING], lr)

    if sched["merge"] == "chunked" and args.chunks == 0 and bench.comm is None and not args.no_calibrate:
        sched = calibrate_chunks(bench, wl, sched, ring, lr)
    m = measure_workload(bench, wl, sched, args.steps, args.warmup, args.repeats, ring, lr,
                         with_alone=(not compact) or args.sweep)
    clocks = sampler.stop(m.get("headline_window")) if sampler else None
    ms = m["headline"]["ms_per_step"]
    value = world * K * P / (ms * 1e-3)
    bpu = path_bytes_per_update(wl, sched)
    if compact:
        del ring
        torch.cuda.empty_cache()
        return {"value": value, "unit": UNIT, "ms_per_step": ms, "ms_min": m["headline"]["min"], "ms_max": m["headline"]["max"],
                "repeats": args.repeats, "steps": args.steps, "gpu_launches_per_step": m["headline"]["launches"] / args.steps,
                "schedule": sched, "bytes_per_update": bpu, "whole_path_gbs": value / world * bpu / 1e9,
                "averaging_hidden_frac": m["hidden"], "kernels_ms_per_step": m["kernels_ms_per_step"],
                "alone": m.get("alone")}

    peak, peak_kind = measured_peak_gbs()
    alone = m["alone"]
    # The dominant kernel is the local step (with the merge folded in under the chunked / fused schedules).
    # Its launches tile the main stream's whole iteration, so its live rate is taken over the timed region
    # itself: algorithmic bytes of one iteration's step launches / median time of one iteration.  Boundaries
    # between launches and the bandwidth the side-stream mean takes all count against it.
    launches_step = m["kernel_launches_per_step"]["local_step"]
    merge_in_step = sched["merge"] in ("chunked", "fused")
    step_b = step_bytes(wl) + ((4.0 / K) / wl["tau"] if merge_in_step else 0.0)
    main_ms = ms if merge_in_step else ms - (m["kernels_ms_per_step"]["merge"] or 0.0)
    step_gbs = K * P * step_b / 1e9 / (main_ms * 1e-3)
    updates_per_launch = K * P / launches_step if launches_step else K * P

    # ---- ablation: the same work with the mean computed inside the step kernel (no side stream)
    ablation = None
    if not args.no_ablation and bench.comm is None:
        eng = bench.make(wl, sched, flags=B.DASGD_FLAG_INLINE_MEAN, snapshot_arrays=False)
        a = bench.repeated(eng, args.steps, args.warmup, min(3, args.repeats), dev_step)
        bytes_a = (step_bytes(wl) * wl["tau"] + 8.0 / K) / wl["tau"]
        ablation = {"schedule": "inline mean: one kernel per iteration, mean summed in registers, no snapshot, "
                                "no side stream (same results; the averaging is no longer asynchronous)",
                    "value": world * K * P / (a["ms_per_step"] * 1e-3), "unit": UNIT, "ms_per_step": a["ms_per_step"],
                    "gpu_launches": a["launches"], "bytes_per_update": bytes_a,
                    "whole_path_gbs": K * P / (a["ms_per_step"] * 1e-3) * bytes_a / 1e9}
        eng.close()
        del eng

    # ---- end to end: gradients start in page-locked host memory every step
    e2e = None
    try:
        if args.no_e2e:
            raise RuntimeError("skipped (--no-e2e)")
        eng = bench.make(wl, sched, host_staging=2)
        hosts = [torch.empty((K, P), dtype=gdt).pin_memory() for _ in range(2)]
        for i, h in enumerate(hosts):
            h.copy_(ring[i])
        probe = torch.empty(1024, dtype=torch.float32).pin_memory()
        torch.cuda.synchronize()
        e2e_steps = max(3, min(args.steps, 20))

        def host_step(e, t):
            e.step_host(hosts[t % 2], lr, probe)

        h = bench.repeated(eng, e2e_steps, 3, min(3, args.repeats), host_step)
        e2e = {"value": world * K * P / (h["ms_per_step"] * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": K * P * (2 if bf16 else 4), "d2h_bytes_per_step": probe.numel() * 4,
               "steps": e2e_steps, "ms_per_step": h["ms_per_step"], "ms_min": h["min"], "ms_max": h["max"],
               "repeats": h["repeats"]}
        eng.close()
        del eng, hosts
    except Exception as ex:  # page-locked memory can be refused on a small host
        e2e = {"value": None, "unit": UNIT, "error": str(ex)[:200]}

    del ring
    torch.cuda.empty_cache()
    others = None
    if rank == 0 and world == 1 and not args.no_others:
        others = other_workloads(args, bench)
    if bench.dist is not None:
        bench.dist.barrier()
        bench.dist.destroy_process_group()
    if rank != 0:
        return None

    cpu = (cpu_baseline(wl) if not args.no_cpu else
           {"value": None, "unit": UNIT, "cores": None, "kind": "oracle", "sample": "skipped (--no-cpu)"})
    kname = "k_local_step_vec (%s%s%s)" % ("bf16 gradients + f32 master" if bf16 else "float32",
                                           ", momentum" if wl["momentum"] else "", ", xi-merge folded in" if merge_in_step else "")
    stall = m.get("stall_ms_per_step")
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "ms_per_step_min": m["headline"]["min"], "ms_per_step_max": m["headline"]["max"],
        "repeats": args.repeats, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 gradients, f32 state" if bf16 else "f32", "data": "synthetic",
        "config": workload_config(wl, name, sched, args.shard, world),
        "clocks": clocks, "e2e": e2e, "gpu_launches": m["headline"]["launches"],
        "roofline": {"bound": "hbm", "kernel": kname,
                     "achieved": step_gbs, "peak": peak, "unit": "GB/s",
                     "frac": step_gbs / peak, "peak_kind": f"of {peak_kind}",
                     "frac_of_8TBs": step_gbs / 8000.0,
                     "algorithmic_bytes_per_update": step_b,
                     "algorithmic_bytes_per_launch": updates_per_launch * step_b,
                     "launches_per_step": launches_step,
                     "avg_launch_ms": main_ms / launches_step if launches_step else None,
                     "timed": "over the timed region: the kernel's launches tile the main stream's iteration, so the "
                              "average launch time is the median iteration time / launches per iteration (launch "
                              "boundaries and the bandwidth taken by the side-stream mean count against the kernel)",
                     "instrumented_ms_per_launch": m["kernels_ms_per_launch"]["local_step"],
                     "instrumented_note": "CUDA events around each launch in a separate pass; with two lanes consecutive "
                                          "launches overlap, so these do not add up to the iteration time",
                     "traffic": profiled_traffic(wl, sched, updates_per_launch),
                     "traffic_note": "ncu dram bytes of one launch of the same shape (reads scale with the updates of a "
                                     "launch; the stores still dirty in L2 at kernel end are a constant); null when the "
                                     "kernels changed since the capture",
                     "alone": alone},
        "kernels_ms_per_launch": m["kernels_ms_per_launch"],
        "kernels_ms_per_step": m["kernels_ms_per_step"],
        "averaging_hidden_frac": m["hidden"],
        "averaging_stall_ms_per_step": stall,
        "averaging_hidden_frac_vs_mean_alone": (1.0 - stall * wl["tau"] / alone["mean"]["ms"])
        if stall is not None and "mean" in alone else None,
        "averaging_hidden_frac_cost": hidden_cost(wl, sched, ms, alone),
        "averaging_hidden_note": "averaging_hidden_frac = 1 - (time streams were blocked waiting for a mean) / (time the mean "
                                 "kernels ran), the paper's notion: the critical path does not stall; a wait's stall is "
                                 "[mean complete] - [waiting stream idle], from CUDA events, when positive.  _vs_mean_alone "
                                 "divides by the mean's time on an idle GPU instead.  _cost = 1 - (cycle time - cycle time "
                                 "of the main-stream kernels alone) / mean kernel alone: on one GPU the mean draws on the "
                                 "same HBM as the local step, so its bytes are not free even though nothing waits for it",
        "bytes_per_update": bpu,
        "whole_path_gbs": value / world * bpu / 1e9,
        "whole_path_frac_of_measured": value / world * bpu / 1e9 / peak,
        "ablation_inline_mean": ablation,
        "other_workloads": others,
        "cpu_baseline": cpu,
    }
    return line


def other_workloads(args, bench):
    """Compact figures for the other configurations (each a short run): the linear-regression size, the
    bfloat16 BERT-large size, two corners of the K x tau x d sweep, and the MLP workload."""
    import copy
    a = copy.copy(args)
    a.warmup, a.repeats, a.sweep = 3, 3, False
    out = {}
    t0 = time.perf_counter()
    for key, wl, steps in (("small_K4_P1024_tau4_d1", dict(WORKLOADS["small"], ring=2), 200),
                           ("sweep_K2_tau1_d1", dict(WORKLOADS["resnet50"], K=2, weight_decay=0.0, ring=2), 20),
                           ("sweep_K32_tau4_d2", dict(WORKLOADS["resnet50"], K=32, tau=4, d=2, weight_decay=0.0, ring=1), 20),
                           ("bert_large_bf16_K4_P335M_tau2_d1", dict(WORKLOADS["bert_large"], ring=1), 20)):
        try:
            a.steps = steps
            out[key] = run_ours(a, wl, key, bench=bench, compact=True)
            out[key].pop("alone", None)
        except Exception as ex:
            out[key] = {"error": str(ex)[:200]}
        torch.cuda.empty_cache()
    try:
        a.steps, a.warmup = 30, 3
        out["mlp_K8_4x4096_tau1_d1"] = mlp_figures(a)
    except Exception as ex:
        out["mlp_K8_4x4096_tau1_d1"] = {"error": str(ex)[:200]}
    torch.cuda.empty_cache()
    out["seconds"] = time.perf_counter() - t0
    return out


def run_sweep(args):
    """The K x tau x d sweep at P = 25.6M float32 (one JSON line per point)."""
    args.no_e2e = args.no_cpu = args.no_others = True
    bench = Bench(args)
    for K in (2, 4, 8, 16, 32):
        for tau in (1, 2, 4):
            for d in (1, 2):
                wl = dict(WORKLOADS["resnet50"], K=K, tau=tau, d=d, weight_decay=0.0, ring=2 if K >= 16 else 4)
                r = run_ours(args, wl, "sweep", bench=bench, compact=True)
                r.update(K=K, tau=tau, d=d)
                if r.get("alone"):
                    r["local_step_alone_gbs"] = r["alone"]["local_step"]["GB/s"]
                    r["mean_alone_gbs"] = r["alone"]["mean"]["GB/s"]
                r.pop("alone", None)
                print(json.dumps(r), flush=True)


def mlp_figures(args):
    """End-to-end workload: K=8 replicas of a 4-layer, 4096-wide bf16 MLP trained against a fixed random
    teacher (batch 256 per worker; forward/backward = batched bf16 matmuls of the GEMM library, on the
    main stream), DaSGD update path with tau=1, d=1.  Here the averaging overlaps real compute."""
    from paper_2006_00441_b200 import binding as B

    K, H, L, batch, lr, tau, d, xi = 8, 4096, 4, 256, 1e-3, 1, 1, 0.25
    net = inputs.TeacherMLP(4, K, H, layers=L, batch=batch, device="cuda", dtype=torch.bfloat16)
    net.precompute_batches(4)
    P = net.P
    flops_per_step = 3 * 2 * K * batch * H * H * L      # forward + two backward GEMMs per layer
    base = B.DASGD_FLAG_ROTATE_SNAPSHOT | B.DASGD_FLAG_FUSE_MERGE | B.DASGD_FLAG_TIMING
    n_chunks = auto_chunks(K, P)
    variants = (("separate_merge", base, 0), ("merge_in_step_kernel", base | B.DASGD_FLAG_FUSE_MERGE_D1, 0),
                ("chunked_pipeline", base | B.DASGD_FLAG_TWO_LANES | B.DASGD_FLAG_TWO_SIDE_STREAMS, n_chunks),
                ("inline_mean", B.DASGD_FLAG_INLINE_MEAN | B.DASGD_FLAG_TIMING, 0))
    out = {"P": P, "n_chunks": n_chunks}
    for name, flags, chunks in variants:
        e = B.DaSGD(K, P, tau, d, xi, 0.9, 0.0, dtype=B.DASGD_BF16_MASTER_F32, flags=flags, order_after_current=False,
                    snapshot_arrays=(name != "inline_mean"), n_chunks=chunks)
        e.set_state(net.student_init())
        g = torch.zeros(K, P, dtype=torch.bfloat16, device="cuda")
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        losses = []
        with torch.cuda.stream(e.main):
            def one(t):
                loss = net.forward_backward(t, e.w_lp, g)
                e.step(g, lr)
                return loss
            for t in range(args.warmup):
                one(t)
            e.sync()
            e.reset_timing()
            l0 = e.launches
            ev[0].record()
            for t in range(args.steps):
                loss = one(args.warmup + t)
                if t in (0, args.steps - 1):
                    losses.append(loss)
            e.main.wait_stream(e.side)
            ev[1].record()
            # forward/backward alone, for the breakdown
            e.sync()
            for t in range(10):
                net.forward_backward(t, e.w_lp, g)
            ev[2].record()
        e.sync()
        torch.cuda.synchronize()
        ms = ev[0].elapsed_time(ev[1]) / args.steps
        ms_fb = ev[1].elapsed_time(ev[2]) / 10
        kt = e.kernel_timing()
        hidden = None
        if kt["mean"][0] and kt["mean"][1] > 0:
            hidden = max(0.0, 1.0 - kt["stall"][1] / kt["mean"][1])
        out[name] = {"value": K * P / (ms * 1e-3), "ms_per_step": ms,
                     "ms_forward_backward": ms_fb, "gemm_tflops": flops_per_step / (ms_fb * 1e-3) / 1e12,
                     "ms_update_path": ms - ms_fb, "gpu_launches_per_step": (e.launches - l0) / args.steps,
                     "averaging_hidden_frac": hidden,
                     "kernels_ms_per_step": {k: v[1] / args.steps for k, v in kt.items()},
                     "loss_first_last": [float(x.mean()) for x in losses]}
        e.close()
        del e, g
        torch.cuda.empty_cache()
    # cost-based figure: what the asynchronous mean adds to the update path beyond the main-stream kernels
    for name in ("separate_merge", "merge_in_step_kernel", "chunked_pipeline"):
        k = out[name]["kernels_ms_per_step"]
        if k["mean"] > 0 and name != "chunked_pipeline":   # two lanes: the per-launch times overlap, no such sum
            out[name]["averaging_hidden_frac_cost"] = 1.0 - (out[name]["ms_update_path"] - k["local_step"] - k["merge"]) / k["mean"]
    return out


def run_mlp(args):
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU implementation")
    r = mlp_figures(args)
    best = min((r[k] for k in ("separate_merge", "merge_in_step_kernel", "chunked_pipeline")), key=lambda x: x["ms_per_step"])
    line = {"metric": METRIC, "value": best["value"], "unit": UNIT, "n_gpus": 1, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": best["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16 weights/gradients/activations, f32 master", "data": "synthetic",
            "config": {"workload": f"mlp: K=8 replicas of a 4-layer 4096-wide bias-free ReLU MLP (P={r['P']}), batch 256 per "
                                   f"worker, teacher-student regression, momentum 0.9, lr 0.001, tau=1, d=1, xi=0.25",
                       "K": 8, "P": r["P"], "tau": 1, "d": 1, "xi": 0.25}}
    line.update(r)
    print(json.dumps(line), flush=True)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--repeats", type=int, default=5, help="timed loops of --steps steps; the median is reported")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet50", choices=sorted(WORKLOADS) + ["mlp"])
    ap.add_argument("--P", type=int, default=0, help="override the workload's parameter count (profiling on a small case)")
    ap.add_argument("--K", type=int, default=0, help="override the number of replicas (sweep)")
    ap.add_argument("--tau", type=int, default=0, help="override the averaging period (sweep)")
    ap.add_argument("--d", type=int, default=-1, help="override the delay (sweep)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-baseline leg")
    ap.add_argument("--no-others", action="store_true", help="skip the short runs of the other configurations")
    ap.add_argument("--no-fuse", action="store_true", help="run the unfused schedule (separate snapshot copy and merge)")
    ap.add_argument("--force-dist", action="store_true",
                    help="initialise the NCCL process group even with one rank (exercises the multi-rank plumbing)")
    ap.add_argument("--no-ablation", action="store_true", help="skip the inline-mean ablation leg")
    ap.add_argument("--lanes", type=int, default=1, help="1: alternate the column ranges between two streams; 0: one stream")
    ap.add_argument("--sides", type=int, default=2, help="2: the means of odd column ranges run on a second side stream; 1: one side stream")
    ap.add_argument("--graph", type=int, default=0, help="1: replay each chunked iteration from a CUDA graph")
    ap.add_argument("--chunks", type=int, default=0,
                    help="column ranges of the pipeline (merge folded into the step kernel); 0: by size "
                         "(ranges of about 18 MiB of weights); 1: off (separate merge kernel)")
    ap.add_argument("--shard", default="replicas", choices=["replicas", "workers"],
                    help="replicas: every GPU runs its own copy of the workload (default).  workers: the K workers of "
                         "every GPU are shards of one K*N-worker job; the partial sums are all-reduced over NCCL")
    ap.add_argument("--no-calibrate", action="store_true",
                    help="take the number of column ranges from the formula without the short trial")
    ap.add_argument("--sweep", action="store_true", help="run the K x tau x d sweep instead (one JSON line per point)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.gpus > 1 and "RANK" not in os.environ and args.impl == "ours":
        # no launcher in the environment: start the ranks here, one per GPU, on the loopback address
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    wl = dict(WORKLOADS.get(args.workload, {}))
    if args.P > 0:
        wl["P"] = args.P
    if args.K > 0:
        wl["K"] = args.K
    if args.tau > 0:
        wl["tau"] = args.tau
    if args.d >= 0:
        wl["d"] = args.d
    if args.workload == "mlp":
        run_mlp(args)
    elif args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args, wl, args.workload)
    else:
        line = run_ours(args, wl, args.workload)
        if line:
            print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
