"""Run and time one configuration of the outer step (and optionally routing).

    python -m paper_2506_10911_b200.run_case --W 16 --n 2 --P 8388608 --theta bf16 --steps 3

Prints one JSON line with device times from the library's own event brackets.
Small cases of this command are what the profiler captures; large ones time
the paper-shaped configurations (1.3B / 6.8B-stage models, worker sweeps).
"""

from __future__ import annotations

import argparse
import json

import torch

from . import build, synth


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--W", type=int, default=16)
    ap.add_argument("--n", type=int, default=2)
    ap.add_argument("--P", type=int, default=1 << 23)
    ap.add_argument("--model", choices=list(synth.MODEL_SHAPES), help="take P from a model shape")
    ap.add_argument("--stage-of", type=int, default=0, help="with --model: P of one of this many stages")
    ap.add_argument("--theta", choices=["f32", "bf16"], default="f32")
    ap.add_argument("--drift", choices=["normal", "student_t3"], default="normal")
    ap.add_argument("--alpha", type=float, default=0.5)
    ap.add_argument("--beta", type=float, default=0.7)
    ap.add_argument("--gamma", type=float, default=0.5)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=1)
    ap.add_argument("--stages", type=int, default=1)
    ap.add_argument("--M", type=int, default=0, help="micro-batches per boundary (0: no routing)")
    ap.add_argument("--E", type=int, default=0, help="elements per micro-batch activation")
    ap.add_argument("--act", choices=["f32", "bf16"], default="bf16")
    ap.add_argument("--divergence", action="store_true", help="also time the replica-divergence metric")
    ap.add_argument("--fast-fill", action="store_true", help="fill state with one uniform pass instead of the "
                    "per-chunk normal/drift recipe (timing only; values do not affect the kernels' time)")
    args = ap.parse_args(argv)

    build.build()
    from . import binding as nolo

    P = args.P
    if args.model:
        P = synth.stage_params(args.model, args.stage_of) if args.stage_of else synth.model_params(args.model)
    stride = synth.padded_stride(P)
    tdt = torch.bfloat16 if args.theta == "bf16" else torch.float32
    need = args.W * stride * (8 + (2 if args.theta == "bf16" else 4))
    free, _ = torch.cuda.mem_get_info()
    if need > free * 0.97:
        print(json.dumps({"skipped": f"needs {need / 1e9:.1f} GB, {free / 1e9:.1f} GB free"}))
        return 0
    dev = torch.device("cuda")
    phi = torch.empty((args.W, stride), dtype=torch.float32, device=dev)
    theta = torch.empty((args.W, stride), dtype=tdt, device=dev)
    delta = torch.empty((args.W, stride), dtype=torch.float32, device=dev)
    if args.fast_fill:
        for w in range(args.W):
            phi[w].uniform_(-0.03, 0.03)
            theta[w].copy_(phi[w])
            delta[w].uniform_(-1e-4, 1e-4)
    else:
        synth.fill_state_(phi, theta, delta, P, 0, args.drift)

    h = nolo.nolo_create(args.W, args.n, P, args.stages, args.alpha, args.beta, args.gamma)
    nolo.nolo_bind_state(h, phi, theta, delta)
    route = args.stages > 1 and args.M > 0 and args.E > 0
    if route:
        adt = torch.bfloat16 if args.act == "bf16" else torch.float32
        K = args.M // args.W
        acts = torch.empty((args.stages - 1, args.W, K, args.E), dtype=adt, device=dev)
        for b in range(args.stages - 1):
            acts[b].normal_()
        out = torch.empty_like(acts)
        nolo.nolo_bind_route(h, args.M, args.E, out)

    def step(k):
        nolo.nolo_outer_step(h, k, k)
        if route:
            nolo.nolo_route(h, k, k, acts)

    for k in range(args.warmup):
        step(k)
    torch.cuda.synchronize()
    nolo.nolo_timing_enable(h, True)
    for k in range(args.steps):
        step(args.warmup + k)
    ms, cnt = nolo.nolo_timing_read(h, nolo.NOLO_KERNEL_OUTER)
    bpp = 20 if args.theta == "bf16" else 24
    res = {"W": args.W, "n": args.n, "P": P, "theta": args.theta, "steps": cnt,
           "outer_ms": ms / max(cnt, 1), "bytes_per_param": bpp,
           "outer_gbs": bpp * args.W * P / (ms / max(cnt, 1) * 1e-3) / 1e9,
           "params_per_s": args.W * P / (ms / max(cnt, 1) * 1e-3)}
    if args.divergence:
        for _ in range(args.steps):
            nolo.nolo_divergence(h)
        dms, dcnt = nolo.nolo_timing_read(h, nolo.NOLO_KERNEL_DIVERGENCE)
        res.update(divergence_ms=dms / max(dcnt, 1),
                   divergence_gbs=4 * args.W * P / (dms / max(dcnt, 1) * 1e-3) / 1e9)
    if route:
        rms, rcnt = nolo.nolo_timing_read(h, nolo.NOLO_KERNEL_ROUTE)
        rbytes = 2 * acts.numel() * acts.element_size()
        res.update(route_ms=rms / max(rcnt, 1), route_bytes=rbytes,
                   route_gbs=rbytes / (rms / max(rcnt, 1) * 1e-3) / 1e9)
    nolo.nolo_destroy(h)
    print(json.dumps(res))
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
