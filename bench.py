#!/usr/bin/env python
"""Benchmark of the DaSGD hot path (local step + snapshot + worker-axis mean + delayed merge).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload resnet50|small]

One "step" is one pass of the whole path over one batch of synthetic gradients: a local step of
all K replicas, the merge that lands on that step, the snapshot and the side-stream mean.
Workload "resnet50": K=8 replicas of a P=25.6M float32 vector, momentum 0.9, weight decay 1e-4,
lr 0.1, tau=1, d=1, xi=0.25.  Prints ONE JSON line (rank 0).

--impl reference times the plain CPU checker under oracle/ on the host cores, on a bounded slice of
the same workload (the path is independent across the parameter index, so a slice is exact).
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


def step_bytes(wl):
    """Algorithmic HBM bytes per replica-parameter of one local-step launch."""
    if wl.get("bf16"):
        return (2 + 4 + 4 + 4 + 4 + 2) if wl["momentum"] else (2 + 4 + 4 + 2)
    return 20 if wl["momentum"] else 12   # read w, (m,) g; write w (, m)



# DRAM traffic of one k_local_step_vec<f32, momentum> launch from an ncu capture on a smaller case
# (K=8, P=4M; dram__bytes_read.sum + dram__bytes_write.sum = 384.0 + 204.4 MB for 32M updates); it grows
# in proportion to K*P.  Valid only while the kernel source is the one that was profiled.
NCU_TRAFFIC = {"kernels_sha256_prefix": "329b3ff5ca6ac696", "bytes_per_update": 588.4e6 / 32.0e6,
               "applies_to": "float32 + momentum"}


def profiled_traffic(wl):
    """Bytes one local-step launch moves through DRAM according to the last ncu capture, or None when
    the kernels have changed since, or the workload is not the profiled variant."""
    import hashlib
    try:
        src = os.path.join(ROOT, "paper_2006_00441_b200", "csrc", "dasgd_kernels.cuh")
        if hashlib.sha256(open(src, "rb").read()).hexdigest()[:16] != NCU_TRAFFIC["kernels_sha256_prefix"]:
            return None
    except OSError:
        return None
    if wl.get("bf16") or not wl["momentum"]:
        return None
    return NCU_TRAFFIC["bytes_per_update"] * wl["K"] * wl["P"]


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# ------------------------------------------------------------------ clocks

class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
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
                ["nvidia-smi", "-i", ident, f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
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
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 7:
                    continue
                try:
                    sm.append(float(f[0])); mx.append(float(f[1]))
                except ValueError:
                    continue
                for nm, v in zip(names, f[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(nm)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out["sm_mhz"] = statistics.median(sm)
            out["sm_max_mhz"] = max(mx)
        out["reasons"] = sorted(reasons)
        out["samples"] = len(sm)
        return out


# ------------------------------------------------------------------ CPU oracle legs

def oracle_throughput(wl, seconds_budget: float, steps: int | None = None, warmup: int = 0):
    """Times the CPU checker on the first P_s parameters of every replica.  Returns a dict."""
    import numpy as np

    import oracle

    K = wl["K"]
    probe = oracle.OracleDaSGD(K, 1, 1, 1, 0.5, omp=True)
    cores = probe.threads
    probe.close()
    # calibrate on a slice too large for the CPU caches, so the rate is the DRAM-bound one
    Pc = min(wl["P"], 2_000_000)
    odt = 1 if wl.get("bf16") else 0

    def host_grad(t, idx):
        g = inputs.grad_block(0, t, K, wl["P"], wl["g_std"], p_index=idx,
                              dtype=torch.bfloat16 if odt else torch.float32)
        return g.view(torch.int16).numpy().view(np.uint16) if odt else g.numpy()

    o = oracle.OracleDaSGD(K, Pc, wl["tau"], wl["d"], wl["xi"], wl["momentum"], wl["weight_decay"], dtype=odt, omp=True)
    o.set_state(inputs.shared_start(0, wl["P"], wl["w_std"], p_index=range(Pc)).numpy())
    g = host_grad(0, range(Pc))
    for _ in range(2):
        o.step(g, wl["lr"])
    t0 = time.perf_counter()
    n_cal = 5
    for _ in range(n_cal):
        o.step(g, wl["lr"])
    rate = K * Pc * n_cal / (time.perf_counter() - t0)  # updates/s, rough
    o.close()
    if steps is None:       # cpu_baseline leg: fixed slice, as many steps as fit the budget
        Ps = min(wl["P"], 2_000_000)
        steps = max(3, min(200, int(seconds_budget * rate / (K * Ps))))
    else:                   # reference arm: the caller fixes the steps, the slice is sized to the budget
        Ps = int(min(wl["P"], 4_000_000, max(1024, seconds_budget * rate / (K * (steps + warmup)))))
    idx = range(Ps)
    o = oracle.OracleDaSGD(K, Ps, wl["tau"], wl["d"], wl["xi"], wl["momentum"], wl["weight_decay"], dtype=odt, omp=True)
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
    return {"value": K * Ps * steps / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {Ps} of {wl['P']} parameters of all {K} replicas, {steps} steps "
                      f"(OpenMP build of the checker, {cores} threads)",
            "seconds": dt, "steps": steps, "P_sample": Ps}


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
        "config": workload_config(wl, name),
        "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")},
        "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(wl, name):
    return {"workload": f"{name}: K={wl['K']} replicas x P={wl['P']} {'bf16 gradients + f32 master' if wl.get('bf16') else 'float32'}, momentum {wl['momentum']}, "
                        f"weight decay {wl['weight_decay']}, lr {wl['lr']}, tau={wl['tau']}, d={wl['d']}, xi={wl['xi']}",
            "K": wl["K"], "P": wl["P"], "tau": wl["tau"], "d": wl["d"], "xi": wl["xi"],
            "l2_policy": "inputs larger than L2 (every step streams all K*P-sized arrays; gradients come from a ring of buffers)",
            "parallelism": "independent replicas of the workload per GPU (no collective on this path)"}


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


def run_ours(args, wl, name):
    from paper_2006_00441_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU implementation")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1 or args.force_dist:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    K, P, lr = wl["K"], wl["P"], wl["lr"]
    bf16 = bool(wl.get("bf16"))
    gdt = torch.bfloat16 if bf16 else torch.float32
    RING = wl.get("ring", 4)
    flags_fused = 0 if args.no_fuse else (B.DASGD_FLAG_ROTATE_SNAPSHOT | B.DASGD_FLAG_FUSE_MERGE)
    seed = 1000 + rank  # every rank runs its own replica of the workload

    def make(flags, host_staging=False):
        e = B.DaSGD(K, P, wl["tau"], wl["d"], wl["xi"], wl["momentum"], wl["weight_decay"], flags=flags,
                    dtype=B.DASGD_BF16_MASTER_F32 if bf16 else B.DASGD_F32,
                    device=local_rank, host_staging=host_staging, order_after_current=False)
        e.set_state(inputs.shared_start(seed, P, wl["w_std"], device="cuda"))
        return e

    ring = [inputs.grad_block(seed, t, K, P, wl["g_std"], device="cuda", dtype=gdt) for t in range(RING)]
    torch.cuda.synchronize()

    def timed_loop(e, steps, warmup, step_fn):
        for t in range(warmup):
            step_fn(e, t)
        e.sync()
        barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0 = e.launches
        with torch.cuda.stream(e.main):
            ev0.record()
        for t in range(steps):
            step_fn(e, warmup + t)
        e.main.wait_stream(e.side)        # the last mean belongs to the timed work
        with torch.cuda.stream(e.main):
            ev1.record()
        e.sync()
        barrier()
        ms, _ = whole_job(ev0.elapsed_time(ev1), 0.0, dist, "cuda")
        return ms, e.launches - l0

    def dev_step(e, t):
        e.step(ring[t % RING], lr)

    # ---- headline: inputs resident in HBM
    eng = make(flags_fused)
    sampler = ClockSampler(local_rank) if rank == 0 else None
    ms, launches = timed_loop(eng, args.steps, args.warmup, dev_step)
    clocks = sampler.stop() if sampler else None
    value = world * K * P * args.steps / (ms * 1e-3)
    eng.close()
    del eng

    # ---- instrumented pass: per-kernel device time and the hidden fraction of the averaging
    eng = make(flags_fused | B.DASGD_FLAG_TIMING)
    for t in range(args.warmup):
        dev_step(eng, t)
    eng.reset_timing()
    n_inst = min(args.steps, 100)
    for t in range(n_inst):
        dev_step(eng, args.warmup + t)
    kt = eng.kernel_timing()
    # the same kernels with nothing else on the GPU (no side-stream mean beside them)
    eng.close()
    del eng
    eng = make(flags_fused | B.DASGD_FLAG_TIMING)
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
    peak, peak_kind = measured_peak_gbs()
    n_step, ms_step = kt["local_step"]
    step_gbs = (K * P * step_bytes(wl) / 1e9) / (ms_step / n_step * 1e-3) if n_step else None
    alone = {}
    for kname, nbytes in (("local_step", K * P * step_bytes(wl)), ("mean", K * P * 4 + P * 4),
                          ("merge", K * P * (10 if bf16 else 8) + P * 4)):
        n_k, ms_k = kt_alone[kname]
        if n_k:
            gbs = nbytes / 1e9 / (ms_k / n_k * 1e-3)
            alone[kname] = {"ms": ms_k / n_k, "GB/s": gbs, "frac": gbs / peak}
    # Hidden fraction of the averaging: every microsecond between the two events that bracket the main
    # stream's wait for a mean counts as stall (that includes the cost of the two events themselves).
    hidden = None
    if kt["mean"][0] and kt["mean"][1] > 0:
        hidden = max(0.0, 1.0 - kt["stall"][1] / kt["mean"][1])

    hidden_cost = None
    if all(k in alone for k in ("local_step", "mean", "merge")):
        tau_, d_ = wl["tau"], wl["d"]
        main_alone = tau_ * alone["local_step"]["ms"] + (alone["merge"]["ms"] if d_ < 2 else 0.0)
        hidden_cost = 1.0 - (ms / args.steps * tau_ - main_alone) / alone["mean"]["ms"]

    # ---- ablation: the same work with the mean computed inside the step kernel (no side stream)
    ablation = None
    if not args.no_ablation:
        eng = B.DaSGD(K, P, wl["tau"], wl["d"], wl["xi"], wl["momentum"], wl["weight_decay"],
                      flags=B.DASGD_FLAG_INLINE_MEAN, dtype=B.DASGD_BF16_MASTER_F32 if bf16 else B.DASGD_F32,
                      device=local_rank, order_after_current=False, snapshot_arrays=False)
        eng.set_state(inputs.shared_start(seed, P, wl["w_std"], device="cuda"))
        ms_a, launches_a = timed_loop(eng, args.steps, args.warmup, dev_step)
        bytes_a = (step_bytes(wl) * wl["tau"] + 8.0 / K) / wl["tau"]
        ablation = {"schedule": "inline mean: one kernel per iteration, mean summed in registers, no snapshot, "
                                "no side stream (same results; the averaging is no longer asynchronous)",
                    "value": world * K * P * args.steps / (ms_a * 1e-3), "unit": UNIT, "ms_per_step": ms_a / args.steps,
                    "gpu_launches": launches_a, "bytes_per_update": bytes_a,
                    "whole_path_gbs": K * P * args.steps / (ms_a * 1e-3) * bytes_a / 1e9}
        eng.close()
        del eng

    # ---- end to end: gradients start in page-locked host memory every step
    e2e = None
    try:
        if args.no_e2e:
            raise RuntimeError("skipped (--no-e2e)")
        eng = make(flags_fused, host_staging=2)
        hosts = [torch.empty((K, P), dtype=gdt).pin_memory() for _ in range(2)]
        for i, h in enumerate(hosts):
            h.copy_(ring[i])
        probe = torch.empty(1024, dtype=torch.float32).pin_memory()
        torch.cuda.synchronize()
        e2e_steps = max(3, min(args.steps, 20))

        def host_step(e, t):
            e.step_host(hosts[t % 2], lr, probe)

        ms_e, _ = timed_loop(eng, e2e_steps, 3, host_step)
        e2e = {"value": world * K * P * e2e_steps / (ms_e * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": K * P * (2 if bf16 else 4), "d2h_bytes_per_step": probe.numel() * 4,
               "steps": e2e_steps, "ms_per_step": ms_e / e2e_steps}
        eng.close()
        del eng, hosts
    except Exception as ex:  # page-locked memory can be refused on a small host
        e2e = {"value": None, "unit": UNIT, "error": str(ex)[:200]}

    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    del ring
    torch.cuda.empty_cache()
    if rank != 0:
        return None

    cpu = (oracle_throughput(wl, seconds_budget=15.0) if not args.no_cpu else
           {"value": None, "unit": UNIT, "cores": None, "kind": "oracle", "sample": "skipped (--no-cpu)"})
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 gradients, f32 state" if bf16 else "f32", "data": "synthetic", "config": workload_config(wl, name),
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
        "roofline": {"bound": "hbm", "kernel": "k_local_step_vec (%s%s)" % ("bf16 gradients + f32 master" if bf16 else "float32",
                                                                ", momentum" if wl["momentum"] else ""),
                     "achieved": step_gbs, "peak": peak, "unit": "GB/s",
                     "frac": (step_gbs / peak) if step_gbs else None, "peak_kind": f"of {peak_kind}",
                     "frac_of_8TBs": (step_gbs / 8000.0) if step_gbs else None,
                     "algorithmic_bytes_per_launch": K * P * step_bytes(wl),
                     "avg_launch_ms": (ms_step / n_step) if n_step else None,
                     "timed": f"CUDA events on the launching stream, instrumented pass of {n_inst} steps; the "
                              "side-stream mean kernel runs beside this kernel and shares HBM with it",
                     "traffic": profiled_traffic(wl),
                     "traffic_note": "ncu dram bytes of a K=8, P=4M launch scaled by K*P; below the algorithmic "
                                     "bytes because the last stores are still dirty in L2 when the kernel ends",
                     "alone": alone},
        "kernels_ms_per_launch": {k: (v[1] / v[0] if v[0] else None) for k, v in kt.items()},
        "averaging_hidden_frac": hidden,
        "averaging_hidden_frac_cost": hidden_cost,
        "averaging_hidden_note": "averaging_hidden_frac: share of the mean kernel's time during which the main stream "
                                 "did not wait for it (the paper's notion: the critical path never stalls).  "
                                 "_cost: 1 - (cycle time - cycle time of the main-stream kernels alone) / mean kernel "
                                 "alone; on one GPU the mean competes with the local step for the same HBM, so its "
                                 "bytes are not free even though nothing waits for it",
        "whole_path_gbs": value / world * path_bytes_per_update(wl) / 1e9,
        "ablation_inline_mean": ablation,
        "cpu_baseline": {k: cpu[k] for k in ("value", "unit", "cores", "kind", "sample")},
    }
    return line


def run_sweep(args):
    """The K x tau x d sweep at P = 25.6M float32 (one JSON line per point), then the bf16 workload."""
    args.no_e2e = args.no_cpu = True
    for K in (2, 4, 8, 16, 32):
        for tau in (1, 2, 4):
            for d in (1, 2):
                wl = dict(WORKLOADS["resnet50"], K=K, tau=tau, d=d, weight_decay=0.0)
                line = run_ours(args, wl, "sweep")
                if line:
                    keep = {k: line[k] for k in ("value", "ms_per_step", "gpu_launches", "averaging_hidden_frac",
                                                 "whole_path_gbs", "kernels_ms_per_launch")}
                    if line.get("ablation_inline_mean"):
                        keep["inline_mean_value"] = line["ablation_inline_mean"]["value"]
                        keep["inline_mean_gbs"] = line["ablation_inline_mean"]["whole_path_gbs"]
                    keep.update(K=K, tau=tau, d=d, local_step_alone_gbs=line["roofline"]["alone"]["local_step"]["GB/s"])
                    print(json.dumps(keep), flush=True)


def run_mlp(args):
    """End-to-end workload: K=8 replicas of a 4-layer, 4096-wide bf16 MLP trained against a fixed random
    teacher (batch 256 per worker; forward/backward = batched bf16 matmuls of the GEMM library, on the
    main stream), DaSGD update path with tau=1, d=1.  Here the averaging overlaps real compute."""
    from paper_2006_00441_b200 import binding as B

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU implementation")
    K, H, L, batch, lr, tau, d, xi = 8, 4096, 4, 256, 1e-3, 1, 1, 0.25
    net = inputs.TeacherMLP(4, K, H, layers=L, batch=batch, device="cuda", dtype=torch.bfloat16)
    net.precompute_batches(4)
    P = net.P
    flops_per_step = 3 * 2 * K * batch * H * H * L      # forward + two backward GEMMs per layer
    out = {}
    for name, flags in (("async", B.DASGD_FLAG_ROTATE_SNAPSHOT | B.DASGD_FLAG_FUSE_MERGE | B.DASGD_FLAG_TIMING),
                        ("inline_mean", B.DASGD_FLAG_INLINE_MEAN | B.DASGD_FLAG_TIMING)):
        e = B.DaSGD(K, P, tau, d, xi, 0.9, 0.0, dtype=B.DASGD_BF16_MASTER_F32, flags=flags, order_after_current=False,
                    snapshot_arrays=(name == "async"))
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
            for t in range(20):
                net.forward_backward(t, e.w_lp, g)
            ev[2].record()
        e.sync()
        torch.cuda.synchronize()
        ms = ev[0].elapsed_time(ev[1]) / args.steps
        ms_fb = ev[1].elapsed_time(ev[2]) / 20
        kt = e.kernel_timing()
        hidden = None
        if kt["mean"][0] and kt["mean"][1] > 0:
            hidden = max(0.0, 1.0 - kt["stall"][1] / kt["mean"][1])
        out[name] = {"value": K * P * args.steps / (ms * args.steps * 1e-3), "ms_per_step": ms,
                     "ms_forward_backward": ms_fb, "gemm_tflops": flops_per_step / (ms_fb * 1e-3) / 1e12,
                     "ms_update_path": ms - ms_fb, "gpu_launches": e.launches - l0, "averaging_hidden_frac": hidden,
                     "kernels_ms_per_launch": {k: (v[1] / v[0] if v[0] else None) for k, v in kt.items()},
                     "loss_first_last": [float(x.mean()) for x in losses]}
        e.close()
        del e, g
        torch.cuda.empty_cache()
    line = {"metric": METRIC, "value": out["async"]["value"], "unit": UNIT, "n_gpus": 1, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": out["async"]["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16 weights/gradients/activations, f32 master", "data": "synthetic",
            "config": {"workload": f"mlp: K={K} replicas of a {L}-layer {H}-wide bias-free ReLU MLP (P={P}), batch {batch} per "
                                   f"worker, teacher-student regression, momentum 0.9, lr {lr}, tau={tau}, d={d}, xi={xi}",
                       "K": K, "P": P, "tau": tau, "d": d, "xi": xi},
            "async": out["async"], "inline_mean": out["inline_mean"]}
    print(json.dumps(line), flush=True)


def path_bytes_per_update(wl):
    """Algorithmic HBM bytes per replica-parameter update of the whole path as bench.py schedules it
    (rotating snapshots, merge folded into a step kernel when d >= 2): tau local steps, the snapshot
    (0 B: no copy), the mean (4 + 4/K B), and the merge (4/K B inside a step kernel when d >= 2, else a
    pass of its own: 8 + 4/K B, + 2 B for the bfloat16 copy)."""
    K, tau, d = wl["K"], wl["tau"], wl["d"]
    per_cycle = step_bytes(wl) * tau + (4.0 + 4.0 / K)
    per_cycle += (4.0 / K) if d >= 2 else (8.0 + 4.0 / K + (2.0 if wl.get("bf16") else 0.0))
    return per_cycle / tau


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet50", choices=sorted(WORKLOADS) + ["mlp"])
    ap.add_argument("--P", type=int, default=0, help="override the workload's parameter count (profiling on a small case)")
    ap.add_argument("--K", type=int, default=0, help="override the number of replicas (sweep)")
    ap.add_argument("--tau", type=int, default=0, help="override the averaging period (sweep)")
    ap.add_argument("--d", type=int, default=-1, help="override the delay (sweep)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-baseline leg")
    ap.add_argument("--no-fuse", action="store_true", help="run the unfused schedule (separate snapshot copy and merge)")
    ap.add_argument("--force-dist", action="store_true",
                    help="initialise the NCCL process group even with one rank (exercises the multi-rank plumbing)")
    ap.add_argument("--no-ablation", action="store_true", help="skip the inline-mean ablation leg")
    ap.add_argument("--sweep", action="store_true", help="run the K x tau x d sweep instead (one JSON line per point)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
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
