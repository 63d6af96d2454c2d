"""Run a few chunkkv_compress_layer calls on one seeded workload, for use under a profiler.

  python -m paper_2502_00299_b200.profile_case --config 2 --iters 3 [--L 32768] [--reuse] [--lane-ctas 18]

Prints CUDA-event timings of the calls; under `ncu` select kernels with -k / -s / -c.
"""
from __future__ import annotations

import argparse
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--L", type=int, default=None)
    ap.add_argument("--budget", type=int, default=None)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--sets", type=int, default=2, help="distinct layer inputs to rotate over")
    ap.add_argument("--reuse", action="store_true", help="gather-only layers (index reuse)")
    ap.add_argument("--lane-ctas", type=int, default=0,
                    help="run the layers through one lane with this CTA budget (0: whole-GPU call)")
    args = ap.parse_args()

    import paper_2502_00299_b200 as ck
    from workloads import CONFIGS, make_layer, scaled

    wl = CONFIGS[args.config]
    if args.L is not None:
        wl = scaled(wl, L=args.L, budget=args.budget or max(wl.w + wl.c, args.L // 10))
    elif args.budget is not None:
        wl = scaled(wl, budget=args.budget)
    dev = lambda b: torch.from_numpy(b.view(np.int16)).cuda().view(torch.bfloat16)
    sets = []
    for i in range(args.sets):
        x = make_layer(wl, layer=i)
        sets.append((dev(x.q_obs), dev(x.K), dev(x.V)))
    lane = None
    if args.lane_ctas > 0:
        lane = ck.Lane(wl.L, wl.Hq, wl.Hkv, wl.d, wl.w, wl.c, max_ctas=args.lane_ctas,
                       stream=torch.cuda.current_stream())
    run = lane.compress_layer if lane is not None else ck.compress_layer
    outs = run(*sets[0], wl.Hq, wl.w, wl.c, wl.budget)
    torch.cuda.synchronize()
    evs = []
    for it in range(args.iters):
        q, K, V = sets[it % args.sets]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        run(q, K, V, wl.Hq, wl.w, wl.c, wl.budget, reuse_idx=outs[2] if args.reuse else None,
            out_K=outs[0], out_V=outs[1], out_idx=outs[2])
        e1.record()
        evs.append((e0, e1))
    torch.cuda.synchronize()
    assert (lane.status() if lane is not None else ck.device_status()) == 0
    print(wl.name, "L", wl.L, "us per call:", [round(a.elapsed_time(b) * 1e3, 1) for a, b in evs])


if __name__ == "__main__":
    main()
