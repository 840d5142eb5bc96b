#!/usr/bin/env python
"""Benchmark of the NoLoCo outer step (+ pipeline routing) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one pass of the whole path over one batch of synthetic state:
nolo_outer_step (subgroup draw + fused Eq. 1-3 update) followed by nolo_route
(route draw + permutation gather of the boundary activations).  The headline
workload is the largest of the paper-shaped configurations that fits the
device: one pipeline-stage shard of the 6.8B decoder (8 of 32 layers,
1.61e9 parameters) x W=8 replicas in subgroups of n=2, float32 phi/delta and
bfloat16 theta (129 GB), with the routing of 32 micro-batches of
4 x 2048 x 4096 bfloat16 activations across the 3 stage boundaries (12.9 GB).
If the device has less free memory the 1.3B model (W=8, n=4, all float32,
126 GB) or the 125M model (W=16, n=2, 20 GB) is taken instead and named in
`config.workload`.  The metric is worker-parameters updated per second (W*P
per outer step).  With N GPUs, N independent replicas run (the path has no
cross-GPU exchange); the job's time is the slowest rank's.  Launched without a
process launcher, `--gpus N` starts the N rank processes itself.

At N=1 the line also carries `configs`: one record per paper-shaped
configuration, per kernel path for large subgroups, and for the routing,
divergence and split-phase kernels, each timed with the library's own CUDA
event brackets around the kernel.

Prints one JSON line on rank 0.
"""

from __future__ import annotations

import argparse
import concurrent.futures
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2506_10911_b200 import replicas, synth  # noqa: E402

METRIC = "outer-step params/sec"
UNIT = "worker-params/s"
ALPHA, BETA, GAMMA = 0.5, 0.7, 0.5
FALLBACK_HBM_GBS = 6650.0
GB = 1e9

# The paper-shaped workloads, largest first.  tokens = sequences x sequence length per micro-batch.
WORKLOADS = [
    dict(name="config 4", W=8, n=2, model="6.8B", stage_of=4, theta="bf16", stages=4, M=32, tokens=4 * 2048,
         text="one of 4 pipeline-stage shards of the 6.8B decoder (8 layers)"),
    dict(name="config 3", W=8, n=4, model="1.3B", stage_of=0, theta="f32", stages=1, M=0, tokens=0,
         text="1.3B decoder flattened"),
    dict(name="config 2", W=16, n=2, model="125M", stage_of=0, theta="bf16", stages=2, M=16, tokens=4 * 1024,
         text="125M decoder flattened"),
]

# DRAM bytes per worker-parameter of the headline kernels from a profiler capture of a small case
# of the same kernel (dram__bytes_read.sum + dram__bytes_write.sum over the worker-parameters of
# the captured launch); traffic grows in proportion to the columns processed.  None = not captured
# since the kernel last changed.
PROFILED_DRAM_BYTES_PER_PARAM = {
    "outer_step_reg_kernel<2,bf16,1>": 2.627498e9 / (16 * 8388608),     # 19.58
    "outer_step_reg_kernel<4,float,1>": 1.553978e9 / (8 * 8388608),      # 23.16
}


def bytes_per_param(theta: str) -> int:
    """Algorithmic bytes per worker-parameter: read phi 4 + theta 4|2 + delta 4, write the same."""
    return 20 if theta == "bf16" else 24


def kernel_name(n: int, theta: str) -> str:
    t = "bf16" if theta == "bf16" else "float"
    if n <= 8:
        items = 4 if n == 1 else (2 if (n == 2 and theta != "bf16") else 1)
        return f"outer_step_reg_kernel<{n},{t},{items}>"
    shape = ("128 threads,128 quads,4 rows" if n <= 12 else "128 threads,64 quads,8 rows" if n <= 24 else
             "256 threads,64 quads,4 rows" if n <= 64 else "256 threads,64 quads,8 rows" if n <= 96 else
             "256 threads,32 quads,4 rows" if n <= 128 else "256 threads,32 quads,8 rows" if n <= 224 else
             "256 threads,16 quads,8 rows" if n <= 640 else "512 threads,16 quads,8 rows")
    return f"outer_step_twopass_kernel<{t},{shape}> (second read of phi from L1/L2)"


def workload_shape(wl):
    d = synth.MODEL_SHAPES[wl["model"]][0]
    P = synth.stage_params(wl["model"], wl["stage_of"]) if wl["stage_of"] else synth.model_params(wl["model"])
    stride = synth.padded_stride(P)
    tb = 2 if wl["theta"] == "bf16" else 4
    E = wl["tokens"] * d
    act_bytes = (wl["stages"] - 1) * wl["M"] * E * 2           # one copy of the boundary activations, bf16
    return dict(P=P, stride=stride, d=d, E=E, K=(wl["M"] // wl["W"] if wl["M"] else 0),
                state_bytes=wl["W"] * stride * (8 + tb), act_bytes=act_bytes)


def pick_workload(free_bytes: int, forced: str | None):
    for wl in WORKLOADS:
        if forced and wl["name"] != forced:
            continue
        sh = workload_shape(wl)
        need = sh["state_bytes"] + 2 * sh["act_bytes"] + (2 << 30)
        if forced or need <= free_bytes:
            return wl, sh
    raise SystemExit(f"no workload fits {free_bytes / GB:.1f} GB of free device memory")


def config_dict(wl, sh, n_gpus):
    route = (f", outer step + routing of {wl['M']} micro-batches of {wl['tokens']}x{sh['d']} bf16 over "
             f"{wl['stages']} stages") if wl["M"] else ", outer step (single stage: no routing)"
    th = "bf16 theta" if wl["theta"] == "bf16" else "fp32 theta"
    return {
        "workload": f"{wl['name']}: W={wl['W']} n={wl['n']} {wl['text']} (P={sh['P']}), fp32 phi/delta, {th}{route}",
        "W": wl["W"], "n": wl["n"], "P": sh["P"], "stages": wl["stages"], "microbatches": wl["M"], "E": sh["E"],
        "alpha": ALPHA, "beta": BETA, "gamma": GAMMA, "replicas": n_gpus,
        "l2": f"state ({sh['state_bytes'] / GB:.1f} GB per replica) is larger than L2; no flush needed",
    }


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clock/throttle samples taken while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "20", "-f", self.path], stdout=subprocess.DEVNULL, stderr=subprocess.DEVNULL)
            time.sleep(0.3)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                   f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# ----------------------------------------------------------------------------
# reference arm / CPU baseline: the oracle, as it stands, on the host cores
# ----------------------------------------------------------------------------

def host_cores() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except Exception:
        return max(1, os.cpu_count() or 1)


def oracle_sample_state(wl, sh, cols: int, seed: int = 0):
    """The first `cols` columns of the workload's state and the matching share of its routed
    activations, as numpy arrays (bfloat16 as uint16 bit patterns)."""
    tdt = torch.bfloat16 if wl["theta"] == "bf16" else torch.float32
    phi, theta, delta = synth.make_state(wl["W"], cols, seed, tdt)
    as_np = lambda x: x.view(torch.int16).numpy().view(np.uint16) if x.dtype == torch.bfloat16 else x.numpy()  # noqa: E731
    out = [as_np(x) for x in (phi, theta, delta)]
    if wl["M"]:
        e_s = max(1, int(sh["E"] * cols / sh["P"]))
        acts = synth.make_acts(wl["stages"] - 1, wl["W"], sh["K"], e_s, 1000 + seed, torch.bfloat16)
        out.append(as_np(acts))
    else:
        out.append(None)
    return out


def oracle_step(wl, state, k: int, threads: int = 1) -> float:
    """One step of the oracle as it stands: outer step, then routing.  With threads > 1 the
    columns are cut into chunks and the same oracle function runs on each chunk in a thread pool
    (the step is independent per column; numpy releases the interpreter lock in its loops)."""
    from oracle import nolo_oracle as O
    W, n = wl["W"], wl["n"]
    dt = O.THETA_BF16 if wl["theta"] == "bf16" else O.THETA_F32
    t0 = time.perf_counter()
    perm = O.draw_groups(k, k, W, n)
    phi, theta, delta, acts = state
    table = O.draw_route(k, k, wl["stages"], W, sh_k(acts)) if acts is not None else None
    if threads <= 1:
        O.outer_step(phi, theta, delta, perm, n, ALPHA, BETA, GAMMA, dt)
        if acts is not None:
            O.route_forward(acts, table)
    else:
        cols = phi.shape[1]
        edges = np.linspace(0, cols, 4 * threads + 1).astype(np.int64)
        jobs = [(int(a), int(b)) for a, b in zip(edges[:-1], edges[1:]) if b > a]
        with concurrent.futures.ThreadPoolExecutor(threads) as pool:
            fut = [pool.submit(O.outer_step, phi[:, a:b], theta[:, a:b], delta[:, a:b], perm, n, ALPHA, BETA, GAMMA, dt)
                   for a, b in jobs]
            if acts is not None:
                e = acts.shape[3]
                ee = np.linspace(0, e, threads + 1).astype(np.int64)
                fut += [pool.submit(O.route_forward, acts[..., int(a):int(b)], table)
                        for a, b in zip(ee[:-1], ee[1:]) if b > a]
            for f in fut:
                f.result()
    return time.perf_counter() - t0


def sh_k(acts) -> int:
    return acts.shape[2]


def c_oracle_step(wl, state, k: int, threads: int) -> float:
    """The same step through the plain-C writing of the oracle (OpenMP over the columns)."""
    from oracle import c_oracle as C
    from oracle import nolo_oracle as O
    W, n = wl["W"], wl["n"]
    C.set_threads(threads)
    t0 = time.perf_counter()
    perm = C.draw_perm(k, k, O.DOMAIN_GROUPS, 0, 0, W)
    phi, theta, delta, acts = state
    C.outer_step(phi, theta, delta, perm, n, ALPHA, BETA, GAMMA, O.THETA_BF16 if wl["theta"] == "bf16" else O.THETA_F32)
    if acts is not None:
        C.route_forward(acts, O.draw_route(k, k, wl["stages"], W, sh_k(acts)))
    return time.perf_counter() - t0


def cpu_baseline(wl, sh, cols: int):
    """One oracle step on the first `cols` columns x all W rows: once on one thread, once with
    the columns spread over all host cores; then the same through the C writing of the oracle."""
    state = oracle_sample_state(wl, sh, cols)
    cores = host_cores()
    t1 = oracle_step(wl, state, 0, 1)
    tc = oracle_step(wl, state, 0, cores) if cores > 1 else t1
    W = wl["W"]
    what = "outer step + routing" if wl["M"] else "outer step"
    rec = {"value": W * cols / tc, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": f"1 step ({what}) on {cols} of {sh['P']} columns x {W} workers, numpy float64: "
                     f"{tc:.1f} s with the columns spread over {cores} threads, {t1:.1f} s on one thread",
           "single_thread": {"value": W * cols / t1, "unit": UNIT, "cores": 1}}
    try:
        c1 = c_oracle_step(wl, state, 0, 1)
        cc = min(c_oracle_step(wl, state, 0, cores) for _ in range(2))
        rec["c_writing"] = {"value": W * cols / cc, "unit": UNIT, "cores": cores, "kind": "oracle (plain C, OpenMP)",
                            "sample": f"the same sample: {cc:.2f} s on {cores} threads, {c1:.2f} s on one",
                            "single_thread": {"value": W * cols / c1, "unit": UNIT, "cores": 1}}
    except Exception as ex:    # no C compiler on the box: the numpy figures stand alone
        rec["c_writing"] = {"value": None, "note": f"{type(ex).__name__}: {ex}"}
    return rec


def run_reference(args):
    rank, _, world = replicas.env_rank()
    if rank != 0:
        return 0
    wl = next(w for w in WORKLOADS if w["name"] == (args.workload or WORKLOADS[0]["name"]))
    sh = workload_shape(wl)
    cores = host_cores()
    probe = oracle_sample_state(wl, sh, 1 << 16)
    t_probe = min(oracle_step(wl, probe, 0, cores) for _ in range(2)) / (1 << 16)   # seconds per column
    budget = args.ref_seconds / max(1, args.steps + args.warmup)
    cols = int(min(1 << 24, max(1 << 12, budget / t_probe)))
    state = oracle_sample_state(wl, sh, cols)
    for k in range(args.warmup):
        oracle_step(wl, state, k, cores)
    t0 = time.perf_counter()
    for k in range(args.steps):
        oracle_step(wl, state, k, cores)
    dt = time.perf_counter() - t0
    W = wl["W"]
    value = W * cols * args.steps / dt
    what = "outer step + routing" if wl["M"] else "outer step"
    sample = (f"each step = 1 oracle step ({what}) on {cols} of {sh['P']} columns x {W} workers "
              f"(numpy float64, columns spread over {cores} threads)")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(wl, sh, world),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# ----------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------

def alloc_state(W, stride, theta, dev):
    tdt = torch.bfloat16 if theta == "bf16" else torch.float32
    return (torch.empty((W, stride), dtype=torch.float32, device=dev),
            torch.empty((W, stride), dtype=tdt, device=dev),
            torch.empty((W, stride), dtype=torch.float32, device=dev))


def stats_record(name, kernel, stats, cnt, nbytes, peak, copy_gbs, **extra):
    gbs = nbytes / (stats["mean"] * 1e-3) / GB if cnt and stats["mean"] > 0 else None
    rec = {"name": name, "kernel": kernel, **extra, "launches_timed": cnt,
           "ms_per_launch": stats["mean"], "ms_per_launch_min": stats["min"], "ms_per_launch_max": stats["max"],
           "bytes_per_launch": nbytes, "gbs": gbs, "frac": gbs / peak if gbs else None,
           "frac_of_same_run_copy": gbs / copy_gbs if gbs and copy_gbs else None}
    return rec


def time_outer_cases(nolo, dev, W, P, theta, variants, peak, copy_gbs, warmup=3, drift="normal",
                     extra_records=False):
    """Allocate and fill one state, then time the outer step for each (name, n, gamma, steps) in
    `variants` on it; returns the records."""
    stride = synth.padded_stride(P)
    need = W * stride * (8 + (2 if theta == "bf16" else 4))
    free = torch.cuda.mem_get_info()[0]
    if need > 0.97 * free:
        return [{"name": v[0], "skipped": f"needs {need / GB:.1f} GB, {free / GB:.1f} GB free"} for v in variants]
    phi, th, delta = alloc_state(W, stride, theta, dev)
    synth.fill_state_(phi, th, delta, P, seed=1, drift=drift)
    recs = []
    for name, n, gamma, steps in variants:
        h = nolo.nolo_create(W, n, P, 1, ALPHA, BETA, gamma)
        nolo.nolo_bind_state(h, phi, th, delta)
        for k in range(warmup):
            nolo.nolo_outer_step(h, k, k)
        torch.cuda.synchronize()
        nolo.nolo_timing_enable(h, True)
        for k in range(steps):
            nolo.nolo_outer_step(h, warmup + k, warmup + k)
        st, cnt = nolo.nolo_timing_stats(h, nolo.NOLO_KERNEL_OUTER)
        recs.append(stats_record(name, kernel_name(n, theta), st, cnt, bytes_per_param(theta) * W * P, peak,
                                 copy_gbs, W=W, n=n, P=P, theta=theta, resident_gb=need / GB,
                                 params_per_s=W * P / (st["mean"] * 1e-3)))
        if extra_records:
            # replica-divergence metric on the same state (read-only, 4 B per worker-parameter)
            for _ in range(steps):
                nolo.nolo_divergence(h)
            st, cnt = nolo.nolo_timing_stats(h, nolo.NOLO_KERNEL_DIVERGENCE)
            recs.append(stats_record(f"{name}: divergence", "divergence_partial_kernel + divergence_final_kernel",
                                     st, cnt, 4 * W * P, peak, copy_gbs, W=W, P=P,
                                     note="read-only pass; the read-only ceiling is above the copy figure"))
            # split-phase step: subgroup means of phi prepared ahead, then the step that uses them
            mean = torch.empty((W // n, stride), dtype=torch.float64, device=dev)
            nolo.nolo_bind_prepared(h, mean)
            for k in range(steps):
                nolo.nolo_outer_prepare(h, 77, k)
                nolo.nolo_outer_step_prepared(h, 77, k)
            sp, cp = nolo.nolo_timing_stats(h, nolo.NOLO_KERNEL_PREPARE)
            so, co = nolo.nolo_timing_stats(h, nolo.NOLO_KERNEL_OUTER)
            recs.append(stats_record(f"{name}: split-phase prepare", "group_mean_kernel", sp, cp,
                                     int((4 + 8 / n) * W * P), peak, copy_gbs, W=W, n=n, P=P,
                                     note="reads phi (4 B), writes float64 subgroup means (8/n B) per "
                                          "worker-parameter"))
            recs.append(stats_record(f"{name}: split-phase step", kernel_name(n, theta) + " with prepared means",
                                     so, co, int((bytes_per_param(theta) + 8 / n) * W * P), peak, copy_gbs,
                                     W=W, n=n, P=P,
                                     note="the fused step's bytes plus the float64 means (8/n B per "
                                          "worker-parameter)"))
            del mean
        nolo.nolo_destroy(h)
    del phi, th, delta
    torch.cuda.empty_cache()
    return recs


def extra_configs(nolo, dev, peak, copy_gbs, args):
    """One record per paper-shaped configuration other than the headline, per large-subgroup
    kernel path, and for the NEXT kernels.  N=1 only."""
    out = []
    run = lambda *a, **kw: out.extend(time_outer_cases(nolo, dev, *a, peak=peak, copy_gbs=copy_gbs, **kw))  # noqa: E731
    run(4, 1 << 20, "f32", [("config 1: W=4 n=2 P=2^20 fp32 (state 50 MB: partly L2-resident)", 2, GAMMA, 20)])
    run(16, synth.model_params("125M"), "bf16", [("config 2: W=16 n=2 125M decoder, bf16 theta", 2, GAMMA, 10)],
        extra_records=True)
    run(8, synth.model_params("1.3B"), "f32",
        [(f"config 3: W=8 n=4 1.3B decoder fp32, gamma={g}", 4, g, 3) for g in (0.0, 0.5)])
    if "config 4" not in args.headline:
        run(8, synth.stage_params("6.8B", 4), "bf16", [("config 4: W=8 n=2 6.8B/4 stage shard, bf16 theta", 2, GAMMA, 3)])
    for W in (8, 32, 128):
        run(W, 1 << 26, "f32", [(f"config 5: W={W} n={n} P=2^26 fp32, Student-t(3) drift", n, GAMMA, 3)
                                for n in (2, 4, 8)], drift="student_t3")
    for n in (9, 16, 32, 64, 96, 128, 192, 256, 512, 1024):
        for theta in ("f32", "bf16"):
            P = max(1 << 16, ((3 << 28) // n) & ~63)           # about 3.2e9 bytes of phi
            run(n, P, theta, [(f"large_n: one subgroup of n=W={n}, P={P}, {theta} theta (DiLoCo mode)", n, GAMMA, 5)])
    return out


# Issue-slot bound of the simulation kernels.  Thread-instructions per log-normal sample, from a
# profiler capture of each kernel (warp instructions x 32 / samples): the straggler kernel spends a
# quarter of a Philox block (ten rounds of two 64 x 64 -> 128-bit products) and half a logarithm,
# square root and sine/cosine pair plus one exponential in float64 per sample; the tree kernel
# computes every block twice (one thread per sibling pair) and walks the tree.  The bound is
# SMs x 4 schedulers x 32 lanes x SM clock / that count.
SIM_THREAD_INSTR_PER_SAMPLE = {"straggler_kernel": 278.0, "tree_allreduce_kernel": 420.0}


def sim_records(nolo):
    """The paper's two latency simulations at Fig. 5's largest size: device time between CUDA
    events around the (synchronous) calls, log-normal samples per second, and the fraction of the
    issue-slot bound."""
    import math
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            sm_hz = float(json.load(f)["sm_max_mhz"]) * 1e6
    except Exception:
        sm_hz = 1.965e9
    sms = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
    slots = sms * 4 * 32 * sm_hz                                  # thread-instructions per second
    out = []
    cases = [("simulation: straggler barrier (Fig. 5b), W=1024 n=2 H=100 T=250, 592 trials", "straggler_kernel",
              lambda: nolo.nolo_sim_straggler(1024, 2, 100, 250, 1.0, math.sqrt(0.5), 592, 0), 592 * 1024 * 100 * 250),
             ("simulation: tree all-reduce vs pair exchange (Fig. 5a), W=1024 sigma=1, 100000 trials",
              "tree_allreduce_kernel", lambda: nolo.nolo_sim_tree_allreduce(1024, 0.0, 1.0, 100_000, 0),
              100_000 * (4 * 1024 - 4))]
    for name, kernel, call, samples in cases:
        call()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        res = call()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        rate = samples / (ms * 1e-3)
        peak = slots / SIM_THREAD_INSTR_PER_SAMPLE[kernel]
        rec = {"name": name, "kernel": kernel, "ms": ms, "samples": samples, "samples_per_s": rate,
               "roofline": {"bound": "alu", "achieved": rate / 1e9, "peak": peak / 1e9, "unit": "G samples/s",
                            "frac": rate / peak, "peak_kind": "issue slots: SMs x 4 schedulers x 32 lanes x SM clock / "
                                                              f"{SIM_THREAD_INSTR_PER_SAMPLE[kernel]:.0f} profiled thread-instructions per sample"}}
        if kernel == "straggler_kernel":
            rec["barrier_over_subgroup"] = res[0] / res[1]
        else:
            rec["tree_over_pair"] = res[0] / nolo.nolo_expected_pair_exchange(0.0, 1.0)
        out.append(rec)
    return out


def measure_e2e(nolo, args, wl, sh, state, acts, acts_out, world, dev):
    """End to end: state and activations in pinned host memory, through the host entry points.
    The full state (>100 GB) cannot be page-locked on the host, so a column slice of it is
    streamed: the first e2e_cols columns of every worker and the same share of every activation.
    Returns (record, note)."""
    phi, theta, delta = state
    W, n, P, E, M, K = wl["W"], wl["n"], sh["P"], sh["E"], wl["M"], sh["K"]
    try:
        import psutil
        host_free = psutil.virtual_memory().available
    except Exception:
        host_free = 32 << 30
    tb = 2 if wl["theta"] == "bf16" else 4
    cols = min(P, args.e2e_cols)
    while cols > (1 << 20) and world * W * cols * (8 + tb) * 1.3 > 0.4 * host_free:
        cols //= 2
    cols &= ~63
    e_s = max(64, (int(E * cols / P) & ~63)) if M else 0
    try:
        hh = nolo.nolo_create(W, n, cols, wl["stages"], ALPHA, BETA, GAMMA)
        nolo.nolo_bind_state(hh, phi, theta, delta)            # same rows, first `cols` columns
        h_state = [torch.empty((W, cols), dtype=x.dtype, pin_memory=True) for x in state]
        for hs, ds in zip(h_state, state):
            hs.copy_(ds[:, :cols])
        if M:
            shape = (wl["stages"] - 1, W, K, e_s)
            d_in = acts.view(-1)[:int(np.prod(shape))].view(shape)
            d_out = acts_out.view(-1)[:int(np.prod(shape))].view(shape)
            h_acts = torch.empty(shape, dtype=acts.dtype, pin_memory=True).copy_(d_in)
            h_out = torch.empty(shape, dtype=acts.dtype, pin_memory=True)
            nolo.nolo_bind_route(hh, M, e_s, d_out)

        def e2e_step(k):
            nolo.nolo_outer_step_host(hh, k, k, *h_state, host_stride=cols)
            if M:
                nolo.nolo_route_host(hh, k, k, h_acts, h_out, d_in)

        e2e_step(0)
        replicas.barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for k in range(args.e2e_steps):
            e2e_step(1 + k)
        torch.cuda.synchronize()
        e2e_ms = (time.perf_counter() - t0) * 1e3
        replicas.barrier()
        j_ms, j_units = replicas.job_time_and_units(e2e_ms, float(W) * cols * args.e2e_steps, dev)
        state_bytes = W * cols * (8 + tb)
        act_bytes = (h_acts.numel() * h_acts.element_size()) if M else 0
        rec = {"value": replicas.throughput(j_units, j_ms), "unit": UNIT,
               "h2d_bytes_per_step": state_bytes + act_bytes, "d2h_bytes_per_step": state_bytes + act_bytes,
               "steps": args.e2e_steps, "ms_per_step": j_ms / args.e2e_steps,
               "slice": f"the first {cols} of {P} columns of all {W} workers and the same share of every "
                        f"activation ({e_s} of {E} elements): the whole state cannot be page-locked on the host",
               "api": "nolo_outer_step_host + nolo_route_host (pinned host buffers, chunked copies "
                      "overlapped with the kernel)"}
        nolo.nolo_destroy(hh)
        return rec, None
    except Exception as ex:   # e.g. not enough page-lockable host memory
        return None, f"{type(ex).__name__}: {ex}"


def run_ours(args):
    from paper_2506_10911_b200 import build
    build.build()
    from paper_2506_10911_b200 import binding as nolo     # fails loudly if the library is missing

    rank, local_rank, world = replicas.env_rank()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    replicas.init("nccl", dev)
    peak, peak_kind = measured_peak()

    # ---- a plain copy of our own in the same run, as context for the roofline fraction
    copy_gbs = None
    try:
        nbytes = 4 << 30
        src = torch.empty(nbytes, dtype=torch.uint8, device=dev).fill_(1)
        dst = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        copy_gbs = nolo.nolo_copy_probe(src, dst, nbytes, 10)
        del src, dst
        torch.cuda.empty_cache()
    except Exception:
        copy_gbs = None

    wl, sh = pick_workload(torch.cuda.mem_get_info()[0], args.workload)
    W, n, P, stride, E, M, K = wl["W"], wl["n"], sh["P"], sh["stride"], sh["E"], wl["M"], sh["K"]
    phi, theta, delta = alloc_state(W, stride, wl["theta"], dev)
    synth.fill_state_(phi, theta, delta, P, seed=rank)
    acts = acts_out = None
    if M:
        acts = synth.make_acts(wl["stages"] - 1, W, K, E, seed=1000 + rank, dtype=torch.bfloat16, device=dev)
        acts_out = torch.empty_like(acts)

    h = nolo.nolo_create(W, n, P, wl["stages"], ALPHA, BETA, GAMMA)
    nolo.nolo_bind_state(h, phi, theta, delta)
    if M:
        nolo.nolo_bind_route(h, M, E, acts_out)

    def step(k):
        nolo.nolo_outer_step(h, k, k)
        if M:
            nolo.nolo_route(h, k, k, acts)

    for k in range(args.warmup):
        step(k)
    torch.cuda.synchronize()
    nolo.nolo_timing_enable(h, True)
    nolo.nolo_timing_read(h, nolo.NOLO_KERNEL_OUTER)
    nolo.nolo_timing_read(h, nolo.NOLO_KERNEL_ROUTE)
    launches0 = nolo.nolo_launch_count(h)
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid).replace("GPU-", ""))
    if rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    replicas.barrier()
    torch.cuda.synchronize()
    e0.record()
    for k in range(args.steps):
        step(args.warmup + k)
    e1.record()
    torch.cuda.synchronize()
    replicas.barrier()
    clocks = sampler.stop() if rank == 0 else None
    local_ms = e0.elapsed_time(e1)
    outer_stats, outer_cnt = nolo.nolo_timing_stats(h, nolo.NOLO_KERNEL_OUTER)
    route_stats, route_cnt = nolo.nolo_timing_stats(h, nolo.NOLO_KERNEL_ROUTE)
    launches = nolo.nolo_launch_count(h) - launches0
    job_ms, job_units = replicas.job_time_and_units(local_ms, float(W) * P * args.steps, dev)
    value = replicas.throughput(job_units, job_ms)

    # ---- backward routing of the same activations (gradients return along the same path)
    back_stats = back_cnt = None
    if M and rank == 0 and world == 1:
        for k in range(5):
            nolo.nolo_route_backward(h, k, k, acts_out, acts)
        back_stats, back_cnt = nolo.nolo_timing_stats(h, nolo.NOLO_KERNEL_ROUTE)
    nolo.nolo_timing_enable(h, False)

    e2e, e2e_note = (None, "skipped") if args.no_e2e else measure_e2e(
        nolo, args, wl, sh, (phi, theta, delta), acts, acts_out, world, dev)

    if rank != 0:
        nolo.nolo_destroy(h)
        return 0

    kname = kernel_name(n, wl["theta"])
    bpp = bytes_per_param(wl["theta"])
    per_launch_ms = outer_stats["mean"]
    achieved = bpp * W * P / (per_launch_ms * 1e-3) / GB
    dram_bpp = PROFILED_DRAM_BYTES_PER_PARAM.get(kname)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": job_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_dict(wl, sh, world),
        "hbm_gbs": achieved, "pct_of_8tbs_nominal": achieved / 8000.0,
        "clocks": clocks,
        "e2e": e2e if e2e is not None else {"value": None, "unit": UNIT, "note": e2e_note or "skipped"},
        "gpu_launches": launches,
        "roofline": {"bound": "hbm", "kernel": kname, "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                     "frac_of_same_run_copy": achieved / copy_gbs if copy_gbs else None,
                     "frac_note": "peak is a plain torch copy measured earlier on this pool; our own one-shot "
                                  "128-bit copy timed in this run is the tighter ceiling (frac_of_same_run_copy)",
                     "traffic": dram_bpp * W * P if dram_bpp else None,
                     "traffic_note": "profiler dram bytes of a small case of this kernel scaled by columns"
                                     if dram_bpp else "not captured since the kernel last changed",
                     "bytes_per_launch": bpp * W * P,
                     "ms_per_launch": per_launch_ms, "ms_per_launch_min": outer_stats["min"],
                     "ms_per_launch_median": outer_stats["median"], "ms_per_launch_max": outer_stats["max"],
                     "launches_timed": outer_cnt,
                     "plain_copy_same_run_gbs": copy_gbs},
    }
    if M:
        rb = 2 * acts.numel() * acts.element_size()
        line["route"] = stats_record("routing, forward, all boundaries", "route_copy16_kernel", route_stats, route_cnt,
                                     rb, peak, copy_gbs)
        if back_stats is not None:
            line["route_backward"] = stats_record("routing, backward, all boundaries", "route_copy16_kernel",
                                                  back_stats, back_cnt, rb, peak, copy_gbs)
    nolo.nolo_destroy(h)
    del phi, theta, delta, acts, acts_out
    torch.cuda.empty_cache()
    if world == 1 and not args.no_configs:
        args.headline = wl["name"]
        headline_rec = stats_record(f"{wl['name']} (the headline workload above): W={W} n={n} {wl['text']}", kname,
                                    outer_stats, outer_cnt, bpp * W * P, peak, copy_gbs, W=W, n=n, P=P,
                                    theta=wl["theta"], resident_gb=sh["state_bytes"] / GB,
                                    params_per_s=W * P / (per_launch_ms * 1e-3))
        line["configs"] = [headline_rec] + extra_configs(nolo, dev, peak, copy_gbs, args)
        line["simulations"] = sim_records(nolo)
    if args.no_cpu_baseline or world > 1:
        line["cpu_baseline"] = None
    else:
        line["cpu_baseline"] = cpu_baseline(wl, sh, args.cpu_cols)
    print(json.dumps(line), flush=True)
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", choices=[w["name"] for w in WORKLOADS], default=None,
                    help="force a workload instead of taking the largest that fits")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--e2e-cols", type=int, default=1 << 26)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the per-configuration records")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-cols", type=int, default=1 << 25)
    ap.add_argument("--ref-seconds", type=float, default=120.0,
                    help="--impl reference: CPU time the whole run (warm-up + steps) is sized for")
    args = ap.parse_args()
    args.warmup = max(3, args.warmup)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # not under a launcher: start the N rank processes ourselves (one per GPU)
        return replicas.launch(args.gpus, [sys.executable, os.path.abspath(__file__), *sys.argv[1:]])
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    raise SystemExit(main())
