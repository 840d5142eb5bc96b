#!/usr/bin/env python
"""Benchmark of the NoLoCo outer step (+ pipeline routing) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one pass of the whole path over one batch of synthetic state:
nolo_outer_step (subgroup draw + fused Eq. 1-3 update) followed by nolo_route
(route draw + permutation gather of the boundary activations).  The workload is
the 125M-parameter decoder flattened per worker, W=16 workers in subgroups of
n=2, float32 phi/delta and bfloat16 theta, with the activations of its
2-stage / 16-replica layout.  The metric is worker-parameters updated per
second (W*P per outer step).  With N GPUs, N independent replicas run (the path
has no cross-GPU exchange); the job's time is the slowest rank's.

Prints one JSON line on rank 0.
"""

from __future__ import annotations

import argparse
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

# Workload: W=16, n=2, 125M decoder (12 layers, d=768, vocab 50k), bf16 theta.
W, N_GROUP = 16, 2
MODEL = "125M"
ALPHA, BETA, GAMMA = 0.5, 0.7, 0.5
STAGES = 2                      # the paper's (DP16, PP2) layout of the small model
MICROBATCH_TOKENS = 4 * 1024    # 4 sequences of 1024 tokens per micro-batch
BYTES_PER_PARAM = 20            # read phi4+theta2+delta4, write phi4+delta4+theta2
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes per worker-parameter of the fused kernel, from the profiler's dram__bytes_read.sum +
# dram__bytes_write.sum on a 1.34 GB case of the same kernel (W=16, n=2, bf16 theta, P=2^23: 2.6283 GB
# for 134 217 728 worker-parameters); traffic is proportional to the columns processed.
PROFILED_DRAM_BYTES_PER_PARAM = 2.6283e9 / (16 * 8388608)


def workload():
    d = synth.MODEL_SHAPES[MODEL][0]
    P = synth.model_params(MODEL)
    return dict(P=P, stride=synth.padded_stride(P), E=MICROBATCH_TOKENS * d, M=W, d=d)


def config_dict(wl, n_gpus):
    return {
        "workload": f"W={W} n={N_GROUP} {MODEL} decoder flattened (P={wl['P']}), fp32 phi/delta, bf16 theta, "
                    f"outer step + routing of {wl['M']} micro-batches of {MICROBATCH_TOKENS}x{wl['d']} bf16 "
                    f"over {STAGES} stages",
        "W": W, "n": N_GROUP, "P": wl["P"], "stages": STAGES, "microbatches": wl["M"], "E": wl["E"],
        "alpha": ALPHA, "beta": BETA, "gamma": GAMMA,
        "replicas": n_gpus,
        "l2": "state (19.7 GB per replica) is larger than L2; no flush needed",
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

def oracle_sample_state(cols: int, seed: int = 0):
    """The first `cols` columns of the workload's state and the matching share of its routed
    activations, as numpy arrays (bfloat16 as uint16 bit patterns)."""
    wl = workload()
    phi, theta, delta = synth.make_state(W, cols, seed, torch.bfloat16)
    e_s = max(1, int(wl["E"] * cols / wl["P"]))
    acts = synth.make_acts(STAGES - 1, W, wl["M"] // W, e_s, 1000 + seed, torch.bfloat16)
    as_np = lambda x: x.view(torch.int16).numpy().view(np.uint16) if x.dtype == torch.bfloat16 else x.numpy()  # noqa: E731
    return [as_np(x) for x in (phi, theta, delta, acts)]


def time_oracle_step(state, k: int) -> float:
    """One step of the oracle as it stands: outer step, then routing."""
    from oracle import nolo_oracle as O
    t0 = time.perf_counter()
    O.outer_step_seeded(state[0], state[1], state[2], k, k, N_GROUP, ALPHA, BETA, GAMMA, O.THETA_BF16)
    O.route_forward(state[3], O.draw_route(k, k, STAGES, W, state[3].shape[2]))
    return time.perf_counter() - t0


def cpu_baseline(cols: int = 1 << 24):
    """One oracle step on the first `cols` columns x all W rows."""
    state = oracle_sample_state(cols)
    dt = time_oracle_step(state, 0)
    return {"value": W * cols / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"1 step (outer step + routing) on {cols} of {workload()['P']} columns x {W} workers "
                      f"(numpy float64, single thread), {dt:.1f} s"}


def run_reference(args):
    rank, _, world = replicas.env_rank()
    if rank != 0:
        return
    wl = workload()
    probe = oracle_sample_state(1 << 14)
    t_probe = min(time_oracle_step(probe, 0) for _ in range(2)) / (1 << 14)   # seconds per column
    budget = 120.0 / max(1, args.steps + args.warmup)
    cols = int(min(1 << 22, max(1 << 12, budget / t_probe)))
    state = oracle_sample_state(cols)
    for k in range(args.warmup):
        time_oracle_step(state, k)
    t0 = time.perf_counter()
    for k in range(args.steps):
        time_oracle_step(state, k)
    dt = time.perf_counter() - t0
    value = W * cols * args.steps / dt
    sample = (f"each step = 1 oracle step (outer step + routing) on {cols} of {wl['P']} columns x {W} workers "
              f"(numpy float64, 1 thread)")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(wl, world),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------

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

    wl = workload()
    P, stride, E, M = wl["P"], wl["stride"], wl["E"], wl["M"]
    K = M // W
    phi = torch.empty((W, stride), dtype=torch.float32, device=dev)
    theta = torch.empty((W, stride), dtype=torch.bfloat16, device=dev)
    delta = torch.empty((W, stride), dtype=torch.float32, device=dev)
    synth.fill_state_(phi, theta, delta, P, seed=rank)
    acts = synth.make_acts(STAGES - 1, W, K, E, seed=1000 + rank, dtype=torch.bfloat16, device=dev)
    acts_out = torch.empty_like(acts)

    h = nolo.nolo_create(W, N_GROUP, P, STAGES, ALPHA, BETA, GAMMA)
    nolo.nolo_bind_state(h, phi, theta, delta)
    nolo.nolo_bind_route(h, M, E, acts_out)

    def step(k):
        nolo.nolo_outer_step(h, k, k)
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
    outer_ms = outer_stats["mean"] * outer_cnt
    route_ms, route_cnt = nolo.nolo_timing_read(h, nolo.NOLO_KERNEL_ROUTE)
    nolo.nolo_timing_enable(h, False)
    launches = nolo.nolo_launch_count(h) - launches0
    job_ms, job_units = replicas.job_time_and_units(local_ms, float(W) * P * args.steps, dev)
    value = replicas.throughput(job_units, job_ms)

    # ---- a plain copy of our own in the same run, as context for the roofline fraction
    copy_gbs = None
    if rank == 0:
        try:
            nbytes = 4 << 30
            src = torch.empty(nbytes, dtype=torch.uint8, device=dev).fill_(1)
            dst = torch.empty(nbytes, dtype=torch.uint8, device=dev)
            copy_gbs = nolo.nolo_copy_probe(src, dst, nbytes, 10)
            del src, dst
        except Exception:
            copy_gbs = None

    # ---- end to end: state and activations in pinned host memory, through the host entry points
    e2e = None
    e2e_note = None
    host_need = world * (W * stride * 10 + 2 * acts.numel() * acts.element_size())
    try:
        import psutil
        host_free = psutil.virtual_memory().available
    except Exception:
        host_free = None
    if not args.no_e2e and host_free is not None and host_need > 0.5 * host_free:
        e2e_note = (f"skipped: page-locking {host_need / 1e9:.0f} GB for {world} replicas would take more than "
                    f"half of the {host_free / 1e9:.0f} GB of free host memory")
    elif not args.no_e2e:
        try:
            h_state = [torch.empty(x.shape, dtype=x.dtype, pin_memory=True) for x in (phi, theta, delta)]
            for hs, ds in zip(h_state, (phi, theta, delta)):
                hs.copy_(ds)
            h_acts = torch.empty(acts.shape, dtype=acts.dtype, pin_memory=True).copy_(acts)
            h_out = torch.empty(acts.shape, dtype=acts.dtype, pin_memory=True)

            def e2e_step(k):
                nolo.nolo_outer_step_host(h, k, k, *h_state, host_stride=stride)
                nolo.nolo_route_host(h, k, k, h_acts, h_out, acts)

            e2e_step(0)
            replicas.barrier()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for k in range(args.e2e_steps):
                e2e_step(1 + k)
            torch.cuda.synchronize()
            e2e_ms = (time.perf_counter() - t0) * 1e3
            replicas.barrier()
            j_ms, j_units = replicas.job_time_and_units(e2e_ms, float(W) * P * args.e2e_steps, dev)
            state_bytes = W * P * (4 + 2 + 4)
            act_bytes = acts.numel() * acts.element_size()
            e2e = {"value": replicas.throughput(j_units, j_ms), "unit": UNIT,
                   "h2d_bytes_per_step": state_bytes + act_bytes, "d2h_bytes_per_step": state_bytes + act_bytes,
                   "steps": args.e2e_steps, "ms_per_step": j_ms / args.e2e_steps,
                   "api": "nolo_outer_step_host + nolo_route_host (pinned host buffers, chunked copies "
                          "overlapped with the kernel)"}
            del h_state, h_acts, h_out
        except Exception as ex:   # e.g. not enough page-lockable host memory
            e2e_note = f"{type(ex).__name__}: {ex}"

    if rank != 0:
        nolo.nolo_destroy(h)
        return

    peak, peak_kind = measured_peak()
    per_launch_ms = outer_ms / max(1, outer_cnt)
    achieved = BYTES_PER_PARAM * W * P / (per_launch_ms * 1e-3) / 1e9
    route_bytes = 2 * acts.numel() * acts.element_size()
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": job_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_dict(wl, world),
        "hbm_gbs": achieved, "pct_of_8tbs_nominal": achieved / 8000.0,
        "clocks": clocks,
        "e2e": e2e if e2e is not None else {"value": None, "unit": UNIT, "note": e2e_note or "skipped"},
        "gpu_launches": launches,
        "roofline": {"bound": "hbm", "kernel": "outer_step_reg_kernel<2,bf16,1>", "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                     "traffic": PROFILED_DRAM_BYTES_PER_PARAM * W * P,
                     "traffic_note": "ncu dram bytes of a 1.34 GB case of this kernel scaled by columns",
                     "bytes_per_launch": BYTES_PER_PARAM * W * P,
                     "ms_per_launch": per_launch_ms, "ms_per_launch_min": outer_stats["min"],
                     "ms_per_launch_median": outer_stats["median"], "ms_per_launch_max": outer_stats["max"],
                     "launches_timed": outer_cnt,
                     "plain_copy_same_run_gbs": copy_gbs},
        "route": {"ms_per_launch": route_ms / max(1, route_cnt), "bytes_per_launch": route_bytes,
                  "achieved_gbs": route_bytes / (route_ms / max(1, route_cnt) * 1e-3) / 1e9 if route_ms else None},
    }
    if args.no_cpu_baseline or world > 1:
        line["cpu_baseline"] = None
    else:
        line["cpu_baseline"] = cpu_baseline(args.cpu_cols)
    nolo.nolo_destroy(h)
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-cols", type=int, default=1 << 24)
    args = ap.parse_args()
    args.warmup = max(3, args.warmup)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
