"""Run the latency simulations of Section 4.3 on the GPU and print one JSON line.

    python -m paper_2506_10911_b200.run_sim tree --W 1024 --sigma 1.0 --trials 20000
    python -m paper_2506_10911_b200.run_sim straggler --W 1024 --n 2 --H 100 --T 250 --trials 148

``tree`` reports the expected binary-tree all-reduce time and its ratio to the
pair exchange (Fig. 5a); ``straggler`` the time to finish T outer iterations
with a global barrier against subgroup waits (Fig. 5b).
"""

from __future__ import annotations

import argparse
import json
import math
import time

import torch

from . import build


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("kind", choices=["tree", "straggler"])
    ap.add_argument("--W", type=int, default=1024)
    ap.add_argument("--n", type=int, default=2)
    ap.add_argument("--H", type=int, default=100)
    ap.add_argument("--T", type=int, default=250)
    ap.add_argument("--mu", type=float, default=None)
    ap.add_argument("--sigma", type=float, default=None)
    ap.add_argument("--trials", type=int, default=148)
    ap.add_argument("--seed", type=int, default=0)
    args = ap.parse_args(argv)
    build.build()
    from . import binding as nolo
    torch.zeros(1, device="cuda")
    if args.kind == "tree":
        mu = 0.0 if args.mu is None else args.mu
        sigma = 1.0 if args.sigma is None else args.sigma
        nolo.nolo_sim_tree_allreduce(args.W, mu, sigma, 16, args.seed)          # warm-up
        t0 = time.perf_counter()
        mean, se = nolo.nolo_sim_tree_allreduce(args.W, mu, sigma, args.trials, args.seed)
        dt = time.perf_counter() - t0
        pair = nolo.nolo_expected_pair_exchange(mu, sigma)
        res = {"kind": "tree", "W": args.W, "mu": mu, "sigma": sigma, "trials": args.trials,
               "mean_time": mean, "standard_error": se, "pair_exchange": pair, "ratio": mean / pair,
               "log2_W": math.log2(args.W), "seconds": dt,
               "samples_per_s": args.trials * (4 * args.W - 4) / dt}
    else:
        mu = 1.0 if args.mu is None else args.mu
        sigma = math.sqrt(0.5) if args.sigma is None else args.sigma
        nolo.nolo_sim_straggler(args.W, args.n, args.H, 1, mu, sigma, 1, args.seed)            # warm-up
        t0 = time.perf_counter()
        b, s, eb, es = nolo.nolo_sim_straggler(args.W, args.n, args.H, args.T, mu, sigma, args.trials, args.seed)
        dt = time.perf_counter() - t0
        res = {"kind": "straggler", "W": args.W, "n": args.n, "H": args.H, "T": args.T, "mu": mu, "sigma": sigma,
               "trials": args.trials, "barrier_time": b, "subgroup_time": s, "ratio": b / s, "seconds": dt,
               "samples_per_s": args.trials * args.W * args.H * args.T / dt}
    print(json.dumps(res))
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
