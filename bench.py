#!/usr/bin/env python
"""Benchmark of the smoothed top-k hot path (forward + VJP) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One step = one pass of the whole path over one batch of the workload: for every
(p, lambda) variant of the workload, tk_fwd_ex (sort, isotonic solve, dual map,
un-permute; row state saved) followed by tk_vjp from that state.  The default
workload is the n = 4096 shape of the 2^26-element sweep (16384 rows, k = 512,
lambda = 1, p in {2, 4/3}): the largest row length the 50 %-of-HBM target is
stated for.  The other workloads (the remaining sweep shapes, MoE router,
class-logit, expert-choice, pruning) are timed after it and reported under
"other_workloads", each with its own roofline fractions and oracle timing.
Inputs are seeded synthetic data, resident
in HBM before the timed region; each (variant, step) uses the next of a ring of
input/output buffer sets whose total size exceeds the L2 cache, so no step
finds its inputs in L2.  The step's launches are captured once per buffer set in
a CUDA graph and replayed, so that the measurement is not bound by Python.

Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2302_01425_b200 import workloads as wl  # noqa: E402

METRIC = "top-k fwd+VJP elements/s"
UNIT = "elements/s"
BYTES_FWD, BYTES_VJP = 8, 12          # algorithmic bytes per element: theta in + out; theta, g in + grad out
L2_BYTES = 126e6
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0         # the 8 TB/s nameplate figure, reported beside the measured copy bandwidth


ROWS_LIMIT = 0


def workload_cases(name: str):
    cases = _workload_cases(name)
    if ROWS_LIMIT:
        import dataclasses
        cases = [dataclasses.replace(c, rows=min(c.rows, ROWS_LIMIT)) for c in cases]
    return cases


def _workload_cases(name: str):
    if name == "moe_router":
        return wl.moe_router_cases()
    if name == "class_logit":
        return [wl.class_logit_case()]
    if name == "expert_choice":
        return [wl.expert_choice_case()]
    if name == "pruning":
        return [wl.pruning_case()]
    if name == "tiny":
        return wl.tiny_cases()[:1]
    if name.startswith("sweep_n"):
        n = int(name[len("sweep_n"):])
        return [c for c in wl.shape_sweep_cases() if c.n == n]
    raise SystemExit(f"unknown workload {name}")


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def kernel_source_hash(sources=None) -> str:
    """Hash of the kernel sources a traffic record depends on: the listed files (paths relative to the
    repository root: the kernel's translation unit and every header it includes), or all of csrc/."""
    h = hashlib.sha256()
    if sources:
        paths = [os.path.join(ROOT, f) for f in sources]
    else:
        csrc = os.path.join(ROOT, "paper_2302_01425_b200", "csrc")
        paths = [os.path.join(csrc, f) for f in sorted(os.listdir(csrc))]
    for path in paths:
        with open(path, "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def recorded_traffic(workload: str, kernel: str):
    """DRAM bytes per launch of the dominant kernel from the committed ncu summary; None when
    absent or taken on different sources of that kernel."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as fh:
            rec = json.load(fh)
        e = rec[workload][kernel]
        if e.get("source_hash") != kernel_source_hash(e.get("sources")):
            return None
        return e["dram_bytes_per_launch"]
    except Exception:
        return None


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-i", str(self.index), "-lms", "100"],
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
        sm, smax, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); smax.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                      "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(smax)),
                       reasons=sorted(reasons), samples=len(sm))
        return out


# ------------------------------------------------------------------ CPU oracle legs
def cpu_model() -> str:
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                return line.split(":", 1)[1].strip()
    except Exception:
        pass
    return "unknown"


def time_oracle(cases, min_seconds: float, max_rows_elements: int = 1 << 22, single_thread: bool = False):
    """Times the oracle (forward + VJP) on a bounded sample of the workload: for each variant
    the leading rows up to max_rows_elements elements; repeated until min_seconds have passed."""
    from oracle import tko
    flags = tko.FLAG_SINGLE_THREAD if single_thread else 0
    inputs = []
    for c in cases:
        rows = max(1, min(c.rows, max_rows_elements // c.n))
        x = c.theta(rows)
        inputs.append((c, x, c.cotangent(x)))
    tko.fwd(inputs[0][1][:1], inputs[0][0].k, inputs[0][0].p, inputs[0][0].lam, inputs[0][0].mode)
    elements = sum(x.size for _, x, _ in inputs)
    reps, t0 = 0, time.perf_counter()
    while True:
        for c, x, g in inputs:
            tko.fwd(x, c.k, c.p, c.lam, c.mode, flags=flags)
            tko.vjp(x, g, c.k, c.p, c.lam, c.mode, flags=flags)
        reps += 1
        dt = time.perf_counter() - t0
        if dt >= min_seconds or reps >= 1000:
            break
    sample = "; ".join(f"{c.name}: first {x.shape[0]} of {c.rows} rows" for c, x, _ in inputs)
    threads = 1 if single_thread else tko.num_threads()
    return elements * reps / dt, dt / reps, threads, f"{reps} pass(es) over [{sample}]"


def oracle_baseline(cases, seconds: float, max_rows_elements: int = 1 << 22):
    """The cpu_baseline object: the oracle on all host cores and on one, on the same bounded sample."""
    v, sec, threads, sample = time_oracle(cases, seconds, max_rows_elements)
    v1, sec1, _, _ = time_oracle(cases, max(0.2 * seconds, 0.5), max_rows_elements // 8, single_thread=True)
    return {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample,
            "ms_per_pass": sec * 1e3, "single_thread_value": v1, "cpu_model": cpu_model()}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cases = workload_cases(args.workload)
    per_step = []
    threads, sample = 1, ""
    for i in range(args.warmup + args.steps):
        v, sec, threads, sample = time_oracle(cases, 0.0, max_rows_elements=1 << 20)
        if i >= args.warmup:
            per_step.append((v, sec))
    value = float(np.mean([v for v, _ in per_step]))
    ms = float(np.mean([s for _, s in per_step])) * 1e3
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "step": "oracle forward + VJP on a bounded sample",
                   "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": sample, "cpu_model": cpu_model()},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------ multi-rank helpers
def max_over_ranks(value: float, device=None) -> float:
    """Slowest rank's time: the job's time when every rank processes its own rows (weak scaling,
    no collective on the data path).  Works on any initialised backend (nccl on GPUs, gloo on CPU)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(elements_per_rank_step: int, steps: int, world: int, ms_total_max: float) -> float:
    """elements/s of the whole job: all ranks' elements over the slowest rank's time."""
    return world * elements_per_rank_step * steps / (ms_total_max * 1e-3)


# ------------------------------------------------------------------ GPU arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="sweep_n4096")
    ap.add_argument("--impl", default="tk", choices=["tk", "reference"])
    ap.add_argument("--no-graph", action="store_true", help="plain launches instead of CUDA graphs")
    ap.add_argument("--no-extra", action="store_true", help="skip the other workloads' summary")
    ap.add_argument("--cpu-seconds", type=float, default=10.0)
    ap.add_argument("--rows", type=int, default=0, help="profiling aid: only the leading ROWS rows of every variant")
    ap.add_argument("--no-e2e", action="store_true", help="profiling aid: skip the host-buffer leg")
    ap.add_argument("--no-clocks", action="store_true", help="profiling aid: no clock sampling (and no "
                    "extra replays to give the sampler time)")
    args = ap.parse_args()
    global ROWS_LIMIT
    ROWS_LIMIT = max(0, args.rows)
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2302_01425_b200 import binding as tk, build

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if local == 0:
        build.build()
    if world > 1:
        dist.barrier()
    tk.load()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    res = measure(args.workload, args.steps, max(args.warmup, 3), dev, tk, torch,
                  graph=not args.no_graph, barrier=barrier, sample_clocks=not args.no_clocks,
                  e2e=not args.no_e2e)
    if args.no_e2e:
        res.update(e2e_ms_total=float("nan"), e2e_steps=0, h2d_bytes_per_step=0, d2h_bytes_per_step=0)
    ms_total = res["ms_total"]
    if world > 1:
        ms_total = max_over_ranks(ms_total, dev)
        res["e2e_ms_total"] = max_over_ranks(res["e2e_ms_total"], dev)

    if rank == 0:
        peak, peak_kind = hbm_peak()
        steps = res["steps"]
        el_step = res["elements_per_step"]
        value = whole_job_value(el_step, steps, world, ms_total)
        dom = res["dominant"]
        achieved = dom["alg_bytes_per_launch"] / (dom["avg_us"] * 1e-6) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
            "warmup": res["warmup"], "ms_per_step": ms_total / steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": dict(res["config"], parallelism=f"rows sharded x{world}, no collective"),
            "rows_per_s": world * res["rows_per_step"] * steps / (ms_total * 1e-3),
            "path_frac_of_hbm_peak": (BYTES_FWD + BYTES_VJP) * value / world / 1e9 / peak,
            "path_frac_of_nominal_8TBps": (BYTES_FWD + BYTES_VJP) * value / world / 1e9 / NOMINAL_HBM_GBS,
            "roofline": {"bound": "hbm", "kernel": dom["name"], "achieved": achieved, "peak": peak,
                         "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak,
                         "frac_of_nominal_8TBps": achieved / NOMINAL_HBM_GBS,
                         "avg_launch_us": dom["avg_us"],
                         "alg_bytes_per_launch": dom["alg_bytes_per_launch"],
                         "traffic": recorded_traffic(args.workload, dom["name"])},
            "kernels": res["kernels"],
            "clocks": res["clocks"],
            "e2e": {"value": world * el_step * res["e2e_steps"] / (res["e2e_ms_total"] * 1e-3),
                    "unit": UNIT, "h2d_bytes_per_step": res["h2d_bytes_per_step"],
                    "d2h_bytes_per_step": res["d2h_bytes_per_step"], "steps": res["e2e_steps"]},
            "gpu_launches": res["launches_per_step"] * steps,
        }
        if ROWS_LIMIT:
            line["config"]["rows_limit"] = ROWS_LIMIT
        if world == 1 and args.cpu_seconds > 0:
            line["cpu_baseline"] = oracle_baseline(workload_cases(args.workload), args.cpu_seconds)
        if world == 1:
            line["solver_paths"] = solver_paths(args.workload, res, dev, tk, torch, peak)
            if not args.no_extra:
                extra = []
                names = ["moe_router", "class_logit", "expert_choice", "pruning"] + \
                        [f"sweep_n{n}" for n in (8, 64, 512, 4096, 32768)]
                for name in names:
                    if name == args.workload:
                        continue
                    try:
                        r = measure(name, 10, 3, dev, tk, torch, graph=(name == "moe_router"), barrier=barrier,
                                    sample_clocks=False, e2e=False)
                        v2 = r["elements_per_step"] * r["steps"] / (r["ms_total"] * 1e-3)
                        d2 = r["dominant"]
                        a2 = d2["alg_bytes_per_launch"] / (d2["avg_us"] * 1e-6) / 1e9
                        entry = {"workload": name, "value": v2, "unit": UNIT,
                                 "ms_per_step": r["ms_total"] / r["steps"],
                                 "path_frac_of_hbm_peak": (BYTES_FWD + BYTES_VJP) * v2 / 1e9 / peak,
                                 "roofline": {"bound": "hbm", "kernel": d2["name"], "achieved": a2, "peak": peak,
                                              "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": a2 / peak,
                                              "frac_of_nominal_8TBps": a2 / NOMINAL_HBM_GBS,
                                              "avg_launch_us": d2["avg_us"],
                                              "alg_bytes_per_launch": d2["alg_bytes_per_launch"]},
                                 "kernels": r["kernels"], "config": r["config"]}
                        entry.update(solver_paths(name, r, dev, tk, torch, peak))
                        if name == "class_logit":
                            # the loss the paper trains that classifier with (k = 3), on the same logits
                            entry["smooth_topk_loss_k3"] = time_topk_loss(name, dev, tk, torch, k=3, peak=peak)
                        if name == "expert_choice":
                            # the same scores stored [tokens, experts]: the operator along the slow axis
                            entry["slow_axis_fwd_vjp"] = time_cols(name, dev, tk, torch, peak)
                        if args.cpu_seconds > 0:
                            entry["cpu_baseline"] = oracle_baseline(workload_cases(name), min(3.0, args.cpu_seconds))
                        extra.append(entry)
                    except tk.TkError as e:
                        extra.append({"workload": name, "unavailable": str(e)})
                line["other_workloads"] = extra
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def solver_paths(name, r, dev, tk, torch, peak):
    """The forward pass of a workload through the other solver paths, reported beside the timed one
    (tk_fwd_ex with the default solver: for phi(x) = x the threshold form, which needs no sort)."""
    out = {}
    cases = workload_cases(name)
    ncase, mode = cases[0].n, cases[0].mode
    vjp_us = r["kernels"][1]["avg_us"] * r["kernels"][1]["launches_per_step"]
    el = r["elements_per_step"]
    if mode != wl.MODE_TOPKMAG and ncase <= 32768:
        # TK_SOLVER_PAV: the keys are sorted (no permutation asked for: keys alone), then the same block solve
        sf = time_solver_forward(name, dev, tk, torch, tk.TK_SOLVER_PAV)
        fwd_us = sum(x["avg_us"] for x in sf)
        out["sorted_path"] = {
            "forward": sf,
            "path_frac_of_hbm_peak": (BYTES_FWD + BYTES_VJP) * el / ((fwd_us + vjp_us) * 1e-6) / 1e9 / peak,
            "note": "tk_fwd_ex(solver=TK_SOLVER_PAV, state saved) + tk_vjp(from state)"}
    if name.startswith("sweep_n"):
        out["dykstra_forward_100_sweeps"] = time_solver_forward(name, dev, tk, torch, tk.TK_SOLVER_DYKSTRA, sweeps=100)
    if name == "expert_choice":     # that experiment ran 10 sweeps of Dykstra
        out["dykstra_forward_10_sweeps"] = time_solver_forward(name, dev, tk, torch, tk.TK_SOLVER_DYKSTRA, sweeps=10)
    if name in ("sweep_n64", "sweep_n4096"):
        # p = 1.5 (q = 3): no closed-form block solve; the library picks the path
        out["general_p_1.5_forward"] = time_solver_forward(name, dev, tk, torch, tk.TK_SOLVER_AUTO, p_override=1.5)
    if name == "sweep_n512":
        # any sorted w (relaxed rank / sort, Sec. 3): a ramp w = (n, .., 1)/n, and w = 1_k through the same kernel
        out["general_w"] = time_general_w(name, dev, tk, torch)
    return out


def time_general_w(workload, dev, tk, torch, launches=3):
    """tk_fwd_w and tk_vjp_w (parallel pool-adjacent-violators, one thread block per row) on the
    workload's rows, p = 2 and p = 4/3."""
    out = []
    for c in workload_cases(workload):
        x = c.theta()
        th = torch.from_numpy(x).to(dev)
        gt = torch.from_numpy(c.cotangent(x)).to(dev)
        y, grad = torch.empty_like(th), torch.empty_like(th)
        ramp = np.arange(c.n, 0, -1, dtype=np.float32) / c.n
        ones_k = np.r_[np.ones(c.k), np.zeros(c.n - c.k)].astype(np.float32)
        for label, w in (("ramp", ramp), ("1_k", ones_k)):
            wt = torch.from_numpy(w).to(dev)
            rec = {"p": round(c.p, 6), "w": label}
            for key, run in (("fwd_us", lambda: tk.tk_fwd_w(th, wt, c.rows, c.n, c.p, c.lam, y)),
                             ("vjp_us", lambda: tk.tk_vjp_w(th, wt, gt, c.rows, c.n, c.p, c.lam, grad))):
                run()
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(launches):
                    run()
                e1.record()
                torch.cuda.synchronize()
                rec[key] = e0.elapsed_time(e1) * 1e3 / launches
            rec["elements_per_s"] = c.elements / ((rec["fwd_us"] + rec["vjp_us"]) * 1e-6)
            out.append(rec)
        del th, gt, y, grad
    return out


def time_solver_forward(workload, dev, tk, torch, solver, sweeps=0, launches=3, p_override=None):
    """Forward pass through another solver path (alternating projections with a fixed number of
    sweeps, or the sort-free exact solver; p_override: another p on the first variant), per variant."""
    out = []
    cases = workload_cases(workload)
    if p_override is not None:
        import dataclasses
        cases = [dataclasses.replace(cases[0], p=p_override)]
    for c in cases:
        th = torch.from_numpy(c.theta()).to(dev)
        y = torch.empty_like(th)
        st = tk.new_state(c.rows, dev) if solver != tk.TK_SOLVER_DYKSTRA else None
        wsb = tk.tk_workspace_bytes(c.rows, c.n, c.k, c.p, c.mode, solver) if solver == tk.TK_SOLVER_DYKSTRA else 0
        ws = torch.empty(wsb, dtype=torch.uint8, device=dev) if wsb else None
        run = lambda: tk.tk_fwd_ex(th, c.rows, c.n, c.k, c.p, c.lam, c.mode, y, solver=solver, sweeps=sweeps,
                                   state_out=st, workspace=ws)
        run()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(launches):
            run()
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / launches
        out.append({"p": round(c.p, 6), "avg_us": us, "elements_per_s": c.elements / (us * 1e-6)})
        del th, y, ws
    return out


def time_cols(workload, dev, tk, torch, peak, launches=10):
    """tk_fwd_cols (state saved) + tk_vjp_cols (from state, transposed theta reused) on the workload's
    matrix stored [n, rows]: two transposes around each pass."""
    c = workload_cases(workload)[0]
    x = np.ascontiguousarray(c.theta().T)
    th = torch.from_numpy(x).to(dev)
    gt = torch.from_numpy(np.ascontiguousarray(c.cotangent(c.theta()).T)).to(dev)
    out, grad = torch.empty_like(th), torch.empty_like(th)
    ws = torch.empty(tk.tk_cols_workspace_bytes(c.n, c.rows), dtype=torch.uint8, device=dev)
    st = tk.new_state(c.rows, dev)

    def run():
        tk.tk_fwd_cols(th, c.n, c.rows, c.rows, c.k, c.p, c.lam, c.mode, out, workspace=ws, state_out=st)
        tk.tk_vjp_cols(None, gt, c.n, c.rows, c.rows, c.k, c.p, c.lam, c.mode, grad, workspace=ws, state=st)
    for _ in range(3):
        run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(launches):
        run()
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / launches
    return {"avg_us": us, "elements_per_s": c.elements / (us * 1e-6),
            "path_frac_of_hbm_peak": (BYTES_FWD + BYTES_VJP) * c.elements / (us * 1e-6) / 1e9 / peak}


def time_topk_loss(workload, dev, tk, torch, k, peak, launches=10):
    """tk_topk_loss (forward pass + reduction pass) on the workload's logits, p = 2 and p = 4/3.
    Algorithmic bytes: theta read once, gradient written once (8 B per element)."""
    out = []
    c = workload_cases(workload)[0]
    th = torch.from_numpy(c.theta()).to(dev)
    tgt = torch.randint(0, c.n, (c.rows,), dtype=torch.int32, device=dev)
    loss = torch.empty((c.rows,), device=dev)
    grad = torch.empty_like(th)
    for p in (2.0, 4.0 / 3.0):
        run = lambda: tk.tk_topk_loss(th, tgt, c.rows, c.n, k, p, c.lam, loss, grad)
        for _ in range(3):
            run()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(launches):
            run()
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / launches
        out.append({"p": round(p, 6), "avg_us": us, "elements_per_s": c.elements / (us * 1e-6),
                    "frac_of_hbm_peak": BYTES_FWD * c.elements / (us * 1e-6) / 1e9 / peak})
    return out


def measure(workload, steps, warmup, dev, tk, torch, graph, barrier, sample_clocks, e2e):
    """Times `steps` steps of the workload on the current device."""
    cases = workload_cases(workload)
    set_bytes = sum(4 * c.elements * 4 for c in cases)           # theta, g, out, grad per variant
    n_groups = max(2, int(np.ceil(2.0 * L2_BYTES / set_bytes)))   # ring of groups > 2 x L2
    n_groups = min(n_groups, 64)
    host = []
    for c in cases:
        x = c.theta()
        host.append((x, c.cotangent(x)))
    groups = []
    for gi in range(n_groups):
        sets = []
        for c, (x, g) in zip(cases, host):
            th = torch.from_numpy(x).to(dev)
            if gi:   # distinct data per ring slot: rows rotated by gi
                th = torch.roll(th, shifts=gi, dims=0).contiguous()
            gt = torch.from_numpy(g).to(dev)
            ws_bytes = tk.tk_workspace_bytes(c.rows, c.n, c.k, c.p, c.mode)
            sets.append({
                "case": c, "theta": th, "g": gt, "out": torch.empty_like(th),
                "grad": torch.empty_like(th), "state": tk.new_state(c.rows, dev),
                "ws": torch.empty(ws_bytes, dtype=torch.uint8, device=dev) if ws_bytes else None})
        groups.append(sets)

    def fwd(s):
        c = s["case"]
        tk.tk_fwd_ex(s["theta"], c.rows, c.n, c.k, c.p, c.lam, c.mode, s["out"], state_out=s["state"],
                     workspace=s["ws"])

    def vjp(s):
        c = s["case"]
        tk.tk_vjp(s["theta"], s["g"], c.rows, c.n, c.k, c.p, c.lam, c.mode, s["grad"], state=s["state"],
                  workspace=s["ws"])

    def step_plain(sets, which="both"):
        for s in sets:
            if which in ("both", "fwd"):
                fwd(s)
            if which in ("both", "vjp"):
                vjp(s)

    stream = torch.cuda.Stream(device=dev)
    runners = {}
    with torch.cuda.stream(stream):
        for _ in range(2):                      # first launches (module load, attribute calls)
            step_plain(groups[0])
        stream.synchronize()
        for which in ("both", "fwd", "vjp"):
            if graph:
                gs = []
                for sets in groups:
                    gobj = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(gobj, stream=stream):
                        step_plain(sets, which)
                    gs.append(gobj)
                runners[which] = [g.replay for g in gs]
            else:
                runners[which] = [(lambda sets=sets, which=which: step_plain(sets, which)) for sets in groups]

        def timed(which, count):
            run = runners[which]
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            barrier()
            e0.record(stream)
            for i in range(count):
                run[i % n_groups]()
            e1.record(stream)
            stream.synchronize()
            barrier()
            return e0.elapsed_time(e1)

        timed("both", warmup)
        sampler = ClockSampler(dev.index if dev.index is not None else 0)
        if sample_clocks:
            sampler.start()
            time.sleep(0.3)
        ms_total = timed("both", steps)
        if sample_clocks and ms_total < 1500:   # keep the GPU under the same load long enough to sample
            reps = int(min(50, 1500 / max(ms_total, 1e-3)))
            for _ in range(reps):
                timed("both", steps)
        clocks = sampler.stop() if sample_clocks else None
        ksteps = max(3, min(steps, 50))
        ms_fwd = timed("fwd", ksteps)
        ms_vjp = timed("vjp", ksteps)

        nvar = len(cases)
        el_step = sum(c.elements for c in cases)
        kernels = [
            {"name": "tk_fwd_ex", "launches_per_step": nvar, "avg_us": ms_fwd * 1e3 / (ksteps * nvar),
             "alg_bytes_per_launch": BYTES_FWD * el_step / nvar},
            {"name": "tk_vjp(state)", "launches_per_step": nvar, "avg_us": ms_vjp * 1e3 / (ksteps * nvar),
             "alg_bytes_per_launch": BYTES_VJP * el_step / nvar},
        ]
        for kx in kernels:
            kx["GBps"] = kx["alg_bytes_per_launch"] / (kx["avg_us"] * 1e-6) / 1e9
        dominant = max(kernels, key=lambda kx: kx["avg_us"] * kx["launches_per_step"])

        out = {
            "ms_total": ms_total, "steps": steps, "warmup": warmup, "elements_per_step": el_step,
            "rows_per_step": sum(c.rows for c in cases), "kernels": kernels, "dominant": dominant,
            "clocks": clocks, "launches_per_step": 2 * nvar,
            "config": {
                "workload": workload,
                "variants": [{"rows": c.rows, "n": c.n, "k": c.k, "p": round(c.p, 6), "lambda": c.lam,
                              "mode": ["topkmask", "topk", "topkmag"][c.mode]} for c in cases],
                "step": "per variant: tk_fwd_ex (state saved) + tk_vjp (from state)",
                "l2": f"ring of {n_groups} buffer groups, {n_groups * set_bytes / 1e6:.0f} MB in total "
                      f"(> L2 {L2_BYTES / 1e6:.0f} MB); every step uses the next group",
                "launch": "CUDA graph replay per step" if graph else "plain launches",
            },
        }
        if e2e:
            # end to end: host buffers in, host buffers out, through the same C ABI calls
            pinned = []
            for c, (x, g) in zip(cases, host):
                pinned.append({"x": torch.from_numpy(x).pin_memory(), "g": torch.from_numpy(g).pin_memory(),
                               "out": torch.empty(x.shape, dtype=torch.float32).pin_memory(),
                               "grad": torch.empty(x.shape, dtype=torch.float32).pin_memory()})

            # The variants of a step are independent calls: they alternate between two streams, so
            # that the device-to-host copies of one overlap the host-to-device copies of the next
            # (the link is full duplex).  Both streams start after, and are joined before, the
            # timing events on the main stream.
            lanes = [torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)]

            def e2e_step(sets):
                for i, (s, h) in enumerate(zip(sets, pinned)):
                    with torch.cuda.stream(lanes[i % 2]):
                        s["theta"].copy_(h["x"], non_blocking=True)
                        s["g"].copy_(h["g"], non_blocking=True)
                        fwd(s)
                        vjp(s)
                        h["out"].copy_(s["out"], non_blocking=True)
                        h["grad"].copy_(s["grad"], non_blocking=True)

            def fork():
                for ln in lanes:
                    ln.wait_stream(stream)

            def join():
                for ln in lanes:
                    stream.wait_stream(ln)

            e2e_steps = max(3, min(steps, 20))
            fork()
            for i in range(3):
                e2e_step(groups[i % n_groups])
            join()
            stream.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            barrier()
            e0.record(stream)
            fork()
            for i in range(e2e_steps):
                e2e_step(groups[i % n_groups])
            join()
            e1.record(stream)
            stream.synchronize()
            barrier()
            out.update(e2e_ms_total=e0.elapsed_time(e1), e2e_steps=e2e_steps,
                       h2d_bytes_per_step=sum(2 * c.elements * 4 for c in cases),
                       d2h_bytes_per_step=sum(2 * c.elements * 4 for c in cases))
    del groups
    torch.cuda.empty_cache()
    return out


if __name__ == "__main__":
    main()
