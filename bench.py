#!/usr/bin/env python
"""Benchmark of the fused AsyncMesh step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME]
    python bench.py --impl reference ...        # the CPU oracle on the same metric

A step is one pass of the whole update path (local AdamW, subset selection,
snapshot, delayed sparse averaging with EMA correction, look-ahead) over every
stage of the mesh.  The metric is replica-coordinate updates per second; the
roofline figure divides the bytes a step cannot avoid moving by the measured
step time.  One JSON line is printed by rank 0.
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

METRIC = "replica_param_updates_per_sec"
UNIT = "replica*param/s"
GRAD_SEED, INIT_SEED, MESH_SEED = 0x6AD5, 0x1217, 0x5EED

def measured_traffic_ratio(kernel_name: str, p: float):
    """DRAM traffic of one steady-state launch relative to its algorithmic bytes, as
    measured with ncu (dram__bytes_read.sum + dram__bytes_write.sum) for the kernel the
    handle actually runs, from the table kept next to the profile summaries
    (profiles/dram_traffic.txt: kernel name | p | ratio | capture).  The captures are
    taken on the small `profile` workload; the kernels are streaming scans whose traffic
    grows with the units processed, so the ratio carries over to any workload that runs
    the same kernel at the same p.  None when the table has no such entry."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    try:
        for line in open(path):
            if line.startswith("#") or "|" not in line:
                continue
            f = [x.strip() for x in line.split("|")]
            if f[0] == kernel_name and abs(float(f[1]) - p) <= 1e-9:
                return float(f[2])
    except (OSError, ValueError, IndexError):
        pass
    return None


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", choices=["native", "reference"], default="native")
    ap.add_argument("--workload", default="llama1b",
                    help="toy | llama125m | llama350m | llama1b | profile | profile8")
    ap.add_argument("--p", type=float, default=None)
    ap.add_argument("--tau", type=int, default=None)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--time-diagnostics", action="store_true",
                    help="also time the consensus-error and EMA-spread reductions (CUDA events)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--flags", type=int, default=0, help="asyncmesh_config.flags (diagnostic)")
    ap.add_argument("--optimizer", choices=["adamw", "nadamw"], default="adamw",
                    help="diagnostic: the paper's own NAdamW instead of the workloads' AdamW")
    return ap.parse_args()


def workload_config(args):
    from paper_2601_22442_b200.layouts import DEFAULT_HP, workloads
    w = dict(workloads()[args.workload])
    hp = dict(DEFAULT_HP)
    if args.p is not None:
        hp["p"] = args.p
    if args.tau is not None:
        w["tau"] = args.tau
    return w, hp


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# ---------------------------------------------------------------------------
# multi-rank plumbing (one process per GPU; no data-path collective: the path
# shards by coordinate range, every rank steps its own shard)
# ---------------------------------------------------------------------------

def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def aggregate_over_ranks(local_ms: float, local_units: float, world: int, device=None):
    """(max step-time over ranks, sum of units over ranks).  Uses the default
    process group when world > 1 (NCCL on GPUs, gloo in the CPU tests)."""
    if world <= 1:
        return local_ms, local_units
    import torch
    import torch.distributed as dist
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    u = torch.tensor([local_units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# ---------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.uuid, self.proc, self.path = uuid, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.uuid, "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
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
                for n, v in zip(names, f[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# ---------------------------------------------------------------------------
# the CPU oracle, timed on a bounded sample of the workload
# ---------------------------------------------------------------------------

def time_oracle(w, hp, steps: int, warmup: int, sample_per_stage: int):
    """Times oracle.step on a coordinate slice of every stage (coordinates are
    independent, so a slice evolves exactly as inside the full vector)."""
    import numpy as np
    import oracle
    import synth_inputs as si
    R, tau = w["R"], w["tau"]
    numel = [min(n, sample_per_stage) for n in w["numel"]]
    base = [(n - m) // 2 for n, m in zip(w["numel"], numel)]   # a slice from the middle
    o = oracle.Oracle(R, numel, p=hp["p"], tau=tau, ema_beta=hp["ema_beta"], lr=hp["lr"],
                      beta1=hp["beta1"], beta2=hp["beta2"], eps=hp["eps"],
                      weight_decay=hp["weight_decay"], seed=MESH_SEED, coord_base=base)
    for s, n in enumerate(numel):
        o.init_params(s, si.init_weights_host(INIT_SEED, s, base[s], n))
    spent = 0.0
    for t in range(1, warmup + steps + 1):
        g = [si.grads_host(GRAD_SEED, t, s, R, base[s], n) for s, n in enumerate(numel)]
        t0 = time.perf_counter()
        o.step(g)
        dt = time.perf_counter() - t0
        if t > warmup:
            spent += dt
    units = float(R) * float(sum(numel)) * steps
    return dict(value=units / spent, seconds=spent, units_per_step=float(R) * sum(numel),
                sample="coordinate slice of %d per stage (%d stages, R=%d), %d timed steps after "
                       "%d warm-up, single thread" % (sample_per_stage, len(numel), R, steps, warmup))


def run_reference(args):
    rank, world, _ = dist_env()
    if rank != 0:
        return 0
    w, hp = workload_config(args)
    warm = max(args.warmup, w["tau"] + 1)
    # sized so that K + W steps stay within a few minutes at ~15 ns per unit
    budget_units = 120.0 / 15e-9 / max(1, args.steps + warm)
    per_stage = int(max(4096, min(1 << 20, budget_units / (w["R"] * len(w["numel"])))))
    r = time_oracle(w, hp, args.steps, warm, per_stage)
    line = {
        "impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT,
        "n_gpus": args.gpus, "steps": args.steps, "warmup": warm,
        "ms_per_step": 1e3 * r["seconds"] / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_dict(args, w, hp),
        "cpu_baseline": {"value": r["value"], "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": r["sample"]},
        "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


def config_dict(args, w, hp):
    return {"workload": args.workload, "R": w["R"], "S": len(w["numel"]),
            "params_per_replica": sum(w["numel"]), "p": hp["p"], "tau": w["tau"],
            "ema_beta": hp["ema_beta"],
            "optimizer": ("NAdamW" if getattr(args, "optimizer", "adamw") == "nadamw" else "AdamW")
            + " lr=3e-4 (0.9,0.95) wd=0.1 eps=1e-8",
            "lookahead_delay": "S-1-stage", "state": "fp32",
            "l2": "inputs larger than L2 (every step streams the whole state)"}


# ---------------------------------------------------------------------------
# the native arm
# ---------------------------------------------------------------------------

def run_native(args):
    import torch
    import torch.distributed as dist
    import synth_inputs as si
    import paper_2601_22442_b200 as pkg

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the native arm has no CPU path")
    if args.warmup < 3:
        args.warmup = 3
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    pkg.load()
    si.build()

    w, hp = workload_config(args)
    R, numel, tau = w["R"], w["numel"], w["tau"]
    warm = max(args.warmup, tau + 2)       # averages are being consumed before timing starts
    stream = torch.cuda.current_stream(dev)
    mesh = pkg.AsyncMesh(R, numel, p=hp["p"], tau=tau, ema_beta=hp["ema_beta"], lr=hp["lr"],
                         beta1=hp["beta1"], beta2=hp["beta2"], eps=hp["eps"],
                         weight_decay=hp["weight_decay"], seed=MESH_SEED + rank, device=local,
                         stream=stream.cuda_stream, flags=args.flags, optimizer=args.optimizer)
    for s, n in enumerate(numel):
        tmp = torch.empty(n, dtype=torch.float32, device=dev)
        si.normal_device(tmp, si.stream_key(INIT_SEED + rank, si.KIND_INIT, 0, s, 0), 0, 0.02)
        mesh.init_params(s, tmp)
        del tmp
    grads = mesh.empty_grads()
    for s, n in enumerate(numel):
        si.grads_device(grads[s], GRAD_SEED + rank, 1, s, n)
    torch.cuda.synchronize(dev)

    for _ in range(warm):
        mesh.step(grads)
    mesh.status()

    # ---- timed region: K steps, inputs resident in HBM ----------------------
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid).replace("GPU-", ""))
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize(dev)
    sampler.start()
    ev[0].record(stream)
    for k in range(args.steps):
        mesh.step(grads)
        ev[k + 1].record(stream)
    torch.cuda.synchronize(dev)
    if world > 1:
        dist.barrier()
    clocks = sampler.stop()
    mesh.status()
    per_step = [ev[k].elapsed_time(ev[k + 1]) for k in range(args.steps)]
    total_ms = ev[0].elapsed_time(ev[-1])
    local_ms = total_ms / args.steps
    units_per_step = float(R) * float(sum(numel))
    min_bytes = mesh.min_bytes_last_step()
    ms, units = aggregate_over_ranks(local_ms, units_per_step, world, dev)
    value = units / (ms * 1e-3)

    kernel_name = mesh.kernel_name()
    diagnostics = None
    if args.time_diagnostics:
        # the two read-only reductions, every stage, device time only
        diagnostics = {}
        for what, fn, per_rc in (("consensus_error", mesh.consensus_error, 4.0),
                                 ("ema_variance", mesh.ema_variance, 4.0)):
            for s in range(len(numel)):
                fn(s)                                   # warm-up
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for s in range(len(numel)):
                fn(s)
            e1.record(stream)
            torch.cuda.synchronize(dev)
            d_ms = e0.elapsed_time(e1)
            gbs = per_rc * units_per_step / (d_ms * 1e-3) / 1e9
            diagnostics[what] = {"ms_all_stages": d_ms, "read_GBs": gbs,
                                 "frac_of_copy_peak": gbs / measured_peak_gbs()[0]}

    # ---- end to end: host gradients in, result out, every step ---------------
    e2e = None
    if not args.no_e2e:
        try:
            host = [torch.empty((R, n), dtype=torch.float32, pin_memory=True) for n in numel]
            for s, n in enumerate(numel):
                host[s].copy_(grads[s][:, :n])
            del grads
            torch.cuda.empty_cache()
            h2d = sum(h.numel() * 4 for h in host)
            last = len(numel) - 1
            mesh.step_host(host)                      # warm-up: allocates the staging buffers
            mesh.consensus_error(last)
            if world > 1:
                dist.barrier()
            torch.cuda.synchronize(dev)
            t0 = time.perf_counter()
            for _ in range(args.e2e_steps):
                mesh.step_host(host)
                mesh.consensus_error(last)            # device -> host: 8 B result + 4 B status
                mesh.status()
            torch.cuda.synchronize(dev)
            e_ms = (time.perf_counter() - t0) * 1e3 / args.e2e_steps
            e_ms, e_units = aggregate_over_ranks(e_ms, units_per_step, world, dev)
            e2e = {"value": e_units / (e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                   "d2h_bytes_per_step": 12, "ms_per_step": e_ms, "steps": args.e2e_steps}
            del host
        except Exception as exc:   # e.g. not enough pinned host memory on this machine
            e2e = {"value": None, "unit": UNIT, "error": str(exc)[:200]}
    mesh.destroy()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    peak, peak_kind = measured_peak_gbs()
    achieved = min_bytes / (local_ms * 1e-3) / 1e9
    traffic = measured_traffic_ratio(kernel_name, hp["p"])
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warm, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32",
        "data": "synthetic (seeded pseudo-normal weights and gradients; one gradient set reused "
                "across timed steps, generated outside the timed region)",
        "config": config_dict(args, w, hp),
        "step_ms": {"min": min(per_step), "median": statistics.median(per_step), "max": max(per_step)},
        "clocks": clocks, "e2e": e2e, "gpu_launches": args.steps, "kernel": kernel_name,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_kind": peak_kind + " copy bandwidth",
                     "frac_of_8TBs": achieved / 8000.0, "min_bytes_per_step": min_bytes,
                     "traffic": None if traffic is None else traffic * min_bytes},
    }
    if diagnostics is not None:
        line["diagnostics"] = diagnostics
    if world == 1 and not args.no_cpu_baseline:
        r = time_oracle(w, hp, steps=8, warmup=tau + 1, sample_per_stage=1 << 19)
        line["cpu_baseline"] = {"value": r["value"], "unit": UNIT, "cores": 1, "kind": "oracle",
                                "sample": r["sample"]}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    args = parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_native(args)


if __name__ == "__main__":
    sys.exit(main())
