#!/usr/bin/env python
"""Benchmark of ChunkKV layer compression on B200 (one process per GPU).

Metric: prefix tokens compressed per second per layer, on the Llama-3-8B 32K KV shape
(Hq 32, Hkv 8, d 128, L 32768, w 32, c 10, budget 3276), seeded synthetic bf16 tensors.

A step compresses the 32 layers of one 32K-token sequence: 32 layer calls
(score -> chunk-sum -> top-k -> gather), cycling over NSETS distinct layer inputs (each 134 MB
of K/V, so consecutive layers never find their K/V in L2). The layers are independent, so the
step keeps `--lanes` of them in flight (chunkkv_pipe_layer, each pipe on its own stream with
its share of the SMs and its row gathers on a side stream; `--mode lane` uses
chunkkv_compress_layer_lane instead). `value` is measured with the step captured in a CUDA graph and
replayed (inputs resident in HBM); the same step launched call by call is reported as `eager`,
the same layers one after another on the whole GPU (chunkkv_compress_layer) as
`roofline_more.single_layer`; `e2e` goes through chunkkv_compress_layer_host with pinned host
buffers, copies inside the timed region.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

METRIC = "prefix_tokens_compressed_per_sec_per_layer"
UNIT = "tokens/s/layer"
NSETS = 4
LAYERS_PER_STEP = 32
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
FALLBACK_BF16_SUSTAINED_TFLOPS = 1400.0
# dram__bytes_read.sum + dram__bytes_write.sum of one cfg2 layer through a lane, from ncu captures
# of both launches (layer kernel + row gather): 8 CTAs 69.6 + 13.5 MB, 18 CTAs 69.5 + 13.5 MB
TRAFFIC_BYTES_PER_LAYER = {8: 83.1e6, 18: 83.0e6}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=("ours", "reference"), default="ours")
    ap.add_argument("--config", type=int, default=2, help="workload table entry (2 = headline)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-long", action="store_true", help="skip the 128K / 64K long-context layer timings")
    ap.add_argument("--lanes", type=int, default=18, help="layers in flight (each on 1/lanes of the SMs)")
    ap.add_argument("--lane-ctas", type=int, default=0, help="CTA budget of a lane (0: SMs // lanes)")
    ap.add_argument("--mode", choices=("pipe", "lane"), default="pipe",
                    help="pipe: chunkkv_pipe_layer (layer kernels back to back, row gathers on side streams); "
                         "lane: chunkkv_compress_layer_lane (one layer at a time per lane)")
    return ap.parse_args()


def measured_bf16_sustained_tflops():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops_sustained"]), "measured"
    except Exception:
        return FALLBACK_BF16_SUSTAINED_TFLOPS, "fallback"


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clock/throttle samples while a timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            time.sleep(0.15)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.05)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in out.strip().splitlines():
            f = [v.strip() for v in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm), "reasons": sorted(reasons)}


def layer_bytes(wl, n_max):
    """Algorithmic bytes of one compute layer: K read once for scoring, q_obs, K/V rows read and
    written by the gather."""
    k_bytes = wl.Hkv * wl.L * wl.d * 2
    q_bytes = wl.Hq * wl.w * wl.d * 2
    g_bytes = 4 * wl.Hkv * n_max * wl.d * 2
    return {"score": k_bytes + q_bytes, "gather": g_bytes, "layer": k_bytes + q_bytes + g_bytes}


# ------------------------------------------------------------------------------------- oracle arm
def time_oracle(wl, x, budget_s: float, max_layers: int = 32):
    """The CPU oracle as it stands, on whole layers of the workload, for about budget_s seconds."""
    from oracle import chunkkv_oracle as ora
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        cores = os.cpu_count() or 1
    t0 = time.perf_counter()
    ora.compress_layer(x.q_obs, x.K, x.V, wl.Hq, wl.Hkv, wl.w, wl.c, wl.budget)
    t1 = time.perf_counter() - t0
    n = int(max(1, min(max_layers, round(budget_s / max(t1, 1e-3)))))
    t0 = time.perf_counter()
    for _ in range(n):
        ora.compress_layer(x.q_obs, x.K, x.V, wl.Hq, wl.Hkv, wl.w, wl.c, wl.budget)
    dt = (time.perf_counter() - t0) / n
    return {"value": wl.L / dt, "unit": UNIT, "cores": int(cores), "kind": "oracle",
            "sample": f"{n} whole layers of {wl.name} (all {wl.Hkv} KV heads), {dt * 1e3:.1f} ms per layer"}


def run_reference(args, wl):
    """--impl reference: the fp64 CPU oracle timed on the host cores, rank 0 only."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import chunkkv_oracle as ora
    from workloads import make_layer
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        cores = os.cpu_count() or 1
    x = make_layer(wl)
    G = wl.Hq // wl.Hkv

    def sample(heads: int):
        ora.compress_layer(x.q_obs[:heads * G], x.K[:heads], x.V[:heads], heads * G, heads, wl.w, wl.c,
                           wl.budget)

    t0 = time.perf_counter(); sample(1); t_head = time.perf_counter() - t0
    total_steps = args.steps + args.warmup
    budget_s = 150.0
    heads = int(max(1, min(wl.Hkv, budget_s / total_steps / max(t_head, 1e-4))))
    for _ in range(args.warmup):
        sample(heads)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        sample(heads)
    dt = time.perf_counter() - t0
    ms_per_step = dt / args.steps * 1e3
    # a step's sample covers `heads` of the Hkv heads of one layer: layer-equivalents = heads / Hkv
    value = (heads / wl.Hkv) * wl.L / (dt / args.steps)
    sample_txt = (f"each step = the oracle on {heads} of {wl.Hkv} KV heads of one {wl.name} layer "
                  f"(L {wl.L}); value scales it to a whole layer")
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "impl": "reference",
        "config": {"workload": wl.name, "Hq": wl.Hq, "Hkv": wl.Hkv, "d": wl.d, "L": wl.L, "w": wl.w,
                   "c": wl.c, "budget": wl.budget},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": int(cores), "kind": "oracle",
                         "sample": sample_txt},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------- CUDA arm
def run_ours(args, wl):
    import torch.distributed as dist

    from paper_2502_00299_b200 import build as _build
    _build.build()
    import paper_2502_00299_b200 as ck
    from paper_2502_00299_b200.sharding import job_throughput, max_over_ranks
    from workloads import CONFIGS, make_layer, scaled

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the library")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    lib = ck.lib
    n_max = ck.out_len(wl.L, wl.w, wl.c, wl.budget)
    nbytes = layer_bytes(wl, n_max)
    # the library allocates nothing: one scratch buffer that covers every shape timed below, set up
    # once, before anything is captured in a graph
    ck.ensure_workspace(wl.L, wl.Hq, wl.Hkv, wl.d, wl.w, wl.c)
    ck.ensure_workspace(wl.L, wl.Hq, wl.Hkv, wl.d, wl.w, 1)
    if not args.no_long and rank == 0:
        for lw in (CONFIGS[4], scaled(CONFIGS[5], L=65536)):
            ck.ensure_workspace(lw.L, lw.Hq, lw.Hkv, lw.d, lw.w, lw.c)

    # ---- inputs: NSETS distinct layers (rank r takes sequence r), resident in HBM
    hosts, sets = [], []
    for i in range(NSETS):
        x = make_layer(wl, layer=i, seq=rank)
        hosts.append(x)
        t = [torch.from_numpy(b.view(np.int16)).to(dev).view(torch.bfloat16) for b in (x.q_obs, x.K, x.V)]
        sets.append((t,))

    # ---- lanes: S layers in flight, each on its own stream with 1/S of the SMs and its own scratch
    n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
    S = max(1, args.lanes)
    lane_ctas = args.lane_ctas if args.lane_ctas > 0 else n_sm // S
    stream = torch.cuda.Stream(device=dev)
    lanes = []
    piped = args.mode == "pipe" and S > 1
    if S > 1:
        for li in range(S):
            cls = ck.Pipe if piped else ck.Lane
            ln = cls(wl.L, wl.Hq, wl.Hkv, wl.d, wl.w, wl.c, max_ctas=lane_ctas, device=dev,
                     stream=stream if li == 0 else None)
            lanes.append(ln)
    lane_streams = [ln.stream for ln in lanes] if lanes else [stream]
    # every layer of a step writes its own output buffers
    lane_outs = []
    for _ in range(LAYERS_PER_STEP):
        o = [torch.empty((wl.Hkv, n_max, wl.d), dtype=torch.bfloat16, device=dev) for _ in range(2)]
        o.append(torch.empty((wl.Hkv, n_max), dtype=torch.int32, device=dev))
        lane_outs.append(o)

    def call_layer(i: int, reuse: bool = False, single: bool = False):
        q, K, V = sets[i % NSETS][0]
        li = 0 if single else i % S
        oK, oV, oI = lane_outs[i]
        if piped and not single and not reuse:
            ln = lanes[li]
            st = lib.chunkkv_pipe_layer(
                ln.handle, q.data_ptr(), K.data_ptr(), V.data_ptr(), wl.L, wl.Hq, wl.Hkv, wl.d, wl.w, wl.c, wl.budget,
                oK.data_ptr(), oV.data_ptr(), oI.data_ptr(), ln.stream.cuda_stream)
        elif piped and not single:
            st = lib.chunkkv_compress_layer(       # gather-only layers need no pipe: spread over the lane streams
                None, K.data_ptr(), V.data_ptr(), wl.L, wl.Hq, wl.Hkv, wl.d, wl.w, wl.c, wl.budget, oI.data_ptr(),
                oK.data_ptr(), oV.data_ptr(), oI.data_ptr(), lanes[li].stream.cuda_stream)
        elif S > 1 and not single:
            ln = lanes[li]
            st = lib.chunkkv_compress_layer_lane(
                None if reuse else q.data_ptr(), K.data_ptr(), V.data_ptr(), wl.L, wl.Hq, wl.Hkv, wl.d, wl.w, wl.c,
                wl.budget, oI.data_ptr() if reuse else None, oK.data_ptr(), oV.data_ptr(), oI.data_ptr(),
                ln.buf.data_ptr(), ln.bytes, ln.max_ctas, ln.stream.cuda_stream)
        else:
            st = lib.chunkkv_compress_layer(
                None if reuse else q.data_ptr(), K.data_ptr(), V.data_ptr(), wl.L, wl.Hq, wl.Hkv, wl.d, wl.w, wl.c,
                wl.budget, oI.data_ptr() if reuse else None, oK.data_ptr(), oV.data_ptr(), oI.data_ptr(),
                stream.cuda_stream)
        if st != 0:
            raise ck.ChunkKVError(st, "chunkkv_compress_layer")

    def issue_step(reuse: bool = False, single: bool = False):
        """One step = LAYERS_PER_STEP layers; lane streams fork from and join back into `stream`."""
        multi = S > 1 and not single
        if multi:
            ev = torch.cuda.Event()
            ev.record(stream)
            for st_ in lane_streams[1:]:
                st_.wait_event(ev)
        for i in range(LAYERS_PER_STEP):
            call_layer(i, reuse, single)
        if multi:
            if piped and not reuse:
                for ln in lanes:
                    ln.join()
            for st_ in lane_streams[1:]:
                ev = torch.cuda.Event()
                ev.record(st_)
                stream.wait_event(ev)

    def step_eager():
        issue_step()

    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
            issue_step()
            issue_step(single=True)
    torch.cuda.synchronize()
    if ck.device_status(stream) != 0 or any(ln.status() != 0 for ln in lanes):
        raise RuntimeError("a kernel reported an abandoned wait during warm-up")

    # ---- the step as a CUDA graph
    def capture(**kw):
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr, stream=stream):
            issue_step(**kw)
        return gr

    graph = capture()
    reuse_graph = capture(reuse=True)
    single_graph = capture(single=True)        # one layer at a time on the whole GPU

    def timed(fn, steps):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        with torch.cuda.stream(stream):
            ev0.record(stream)
            for _ in range(steps):
                fn()
            ev1.record(stream)
        barrier()
        return ev0.elapsed_time(ev1)

    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
            graph.replay()
            reuse_graph.replay()
            single_graph.replay()
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        gpu_id = str(local_rank)
    sampler = ClockSampler(gpu_id)
    sampler.start()
    ms_total = timed(graph.replay, args.steps)
    clocks = sampler.stop()
    tokens_local = args.steps * LAYERS_PER_STEP * wl.L
    value, ms_max = job_throughput(tokens_local, ms_total, dev)
    ms_per_step = ms_max / args.steps
    ms_layer = ms_per_step / LAYERS_PER_STEP

    # ---- the same step, call by call (no graph); gather-only (index reuse) layers; one layer at a time
    eager_steps = max(3, min(args.steps, 100))
    ms_eager = max_over_ranks(timed(step_eager, eager_steps), dev) / eager_steps
    ms_reuse = max_over_ranks(timed(reuse_graph.replay, eager_steps), dev) / eager_steps / LAYERS_PER_STEP
    ms_single = max_over_ranks(timed(single_graph.replay, eager_steps), dev) / eager_steps / LAYERS_PER_STEP

    # ---- per-kernel durations (CUDA events around every kernel, on the launching stream)
    ck.profile_enable(True)
    prof_steps = max(3, min(args.steps, 30))
    timed(lambda: issue_step(single=True), prof_steps)      # one layer at a time: each kernel has the GPU to itself
    ms_slot, n_slot = ck.profile_read()
    ck.profile_enable(False)
    names = ("score", "finalize", "select", "gather")
    per_kernel = {n: {"launches": c, "avg_us": (m / c * 1e3) if c else None, "total_ms": m}
                  for n, m, c in zip(names, ms_slot, n_slot)}
    tot = sum(ms_slot) or 1.0
    for n, m in zip(names, ms_slot):
        per_kernel[n]["share"] = m / tot

    peak, peak_src = measured_hbm_peak()
    score_us = per_kernel["score"]["avg_us"] or float("nan")
    fused = per_kernel["gather"]["launches"] == 0          # the whole layer ran as one kernel
    split = S > 1 and 2 * lane_ctas <= n_sm               # a lane's layer = layer kernel + row-gather launch
    launches_per_layer = 2 if (piped or split) else 1           # layer kernel + row gather
    # The timed region holds nothing but the launches of LAYERS_PER_STEP layers per step, S of them
    # in flight at a time on disjoint SM sets, so the duration a launch accounts for is the region
    # divided by the layers; algorithmic bytes per layer over that is what HBM sustains.
    achieved = nbytes["layer"] / (ms_layer * 1e-3) / 1e9
    if piped:
        kernel_name = ("score_kernel<FUSED> on %d CTAs (score + chunk sums + finalize + select) on the pipe's main stream + "
                       "gather_kernel (row gather in CTAs spread over all SMs) on its side stream: the two launches of a "
                       "layer in a pipe" % lane_ctas)
    elif split:
        kernel_name = ("score_kernel<FUSED> on %d CTAs (score + chunk sums + finalize + select) + gather_kernel "
                       "(row gather in CTAs spread over all SMs): the two launches of a layer in a lane" % lane_ctas)
    else:
        kernel_name = "score_kernel<FUSED> (score + chunk sums + finalize + select + gather in one launch)"
    roofline = {"kernel": kernel_name, "bound": "hbm", "achieved": achieved, "peak": peak,
                "peak_source": peak_src, "unit": "GB/s", "frac": achieved / peak,
                "traffic": TRAFFIC_BYTES_PER_LAYER.get(lane_ctas) if ((split or piped) and args.config == 2) else None,
                "algorithmic_bytes_per_launch": nbytes["layer"], "avg_launch_us": ms_layer * 1e3,
                "launches_in_flight": S,
                "isolated_launch_us": score_us,
                "isolated_frac": nbytes["layer"] / (score_us * 1e-6) / 1e9 / peak,
                "note": "avg_launch_us = CUDA-event time of the timed region / layers launched in it "
                        f"({S} layers in flight on disjoint SM sets, nothing else in the region); "
                        "isolated_* = the whole-GPU layer kernel timed alone, one layer at a time; "
                        "traffic = DRAM bytes of one layer's launches from an ncu capture (cold L2)"}
    layer_gbs = nbytes["layer"] / (ms_layer * 1e-3) / 1e9
    gather_us = per_kernel["gather"]["avg_us"]                    # None when the layer kernel is fused
    extra_roof = {
        "layer_throughput": {"algorithmic_bytes": nbytes["layer"], "us_per_layer": ms_layer * 1e3, "GB/s": layer_gbs,
                             "frac_of_measured_peak": layer_gbs / peak, "frac_of_8TBs": layer_gbs / NOMINAL_HBM_GBS,
                             "lanes": S},
        "single_layer": {"algorithmic_bytes": nbytes["layer"], "us": ms_single * 1e3,
                         "GB/s": nbytes["layer"] / (ms_single * 1e-3) / 1e9,
                         "frac_of_measured_peak": nbytes["layer"] / (ms_single * 1e-3) / 1e9 / peak,
                         "note": "layers one after another, each on all SMs"},
        "gather_kernel": None if not gather_us else {
            "algorithmic_bytes": nbytes["gather"], "us": gather_us,
            "GB/s": nbytes["gather"] / (gather_us * 1e-6) / 1e9,
            "frac_of_measured_peak": nbytes["gather"] / (gather_us * 1e-6) / 1e9 / peak},
        "reuse_layer": {"algorithmic_bytes": nbytes["gather"], "us": ms_reuse * 1e3,
                        "GB/s": nbytes["gather"] / (ms_reuse * 1e-3) / 1e9,
                        "frac_of_measured_peak": nbytes["gather"] / (ms_reuse * 1e-3) / 1e9 / peak},
    }

    # ---- variants next to the hot path: token-level selection (c = 1) and the index-similarity diagnostic
    def time_calls(fn, n=30):
        for _ in range(3):
            fn()
        return timed(lambda: [fn() for _ in range(n)], 1) / n * 1e3      # us per call

    n_max1 = ck.out_len(wl.L, wl.w, 1, wl.budget)
    o1 = [torch.empty((wl.Hkv, n_max1, wl.d), dtype=torch.bfloat16, device=dev) for _ in range(2)]
    o1.append(torch.empty((wl.Hkv, n_max1), dtype=torch.int32, device=dev))
    calls = [0]

    def token_level_layer():
        q, K, V = sets[calls[0] % NSETS][0]
        calls[0] += 1
        st = lib.chunkkv_compress_layer(q.data_ptr(), K.data_ptr(), V.data_ptr(), wl.L, wl.Hq, wl.Hkv, wl.d, wl.w, 1,
                                        wl.budget, None, o1[0].data_ptr(), o1[1].data_ptr(), o1[2].data_ptr(),
                                        stream.cuda_stream)
        if st != 0:
            raise ck.ChunkKVError(st, "chunkkv_compress_layer (c = 1)")

    with torch.cuda.stream(stream):
        us_token = time_calls(token_level_layer)
        ia, ib = lane_outs[0][2], lane_outs[1][2]
        us_jac = time_calls(lambda: ck.jaccard(ia, ib, stream=stream))
    bytes1 = layer_bytes(wl, n_max1)["layer"]
    extra_roof["token_level_layer"] = {"c": 1, "algorithmic_bytes": bytes1, "us": us_token,
                                       "GB/s": bytes1 / (us_token * 1e-6) / 1e9,
                                       "frac_of_measured_peak": bytes1 / (us_token * 1e-6) / 1e9 / peak,
                                       "note": "chunkkv_compress_layer with c = 1, one layer at a time on all SMs"}
    extra_roof["jaccard"] = {"us": us_jac, "note": "chunkkv_jaccard on the kept indices of two layers "
                                                   f"([{wl.Hkv}, {n_max}] int32 each; latency-bound, includes the binding's two small allocations)"}

    # ---- the long-context shapes (256 score rows per KV head: bound by exponentials and the tensor
    #      pipe rather than by HBM), one layer at a time on the whole GPU
    if not args.no_long and rank == 0:
        tf_peak, tf_src = measured_bf16_sustained_tflops()
        sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
        long_rows = {}
        for name, lw in (("cfg4_128k", CONFIGS[4]), ("cfg5_longest_64k", scaled(CONFIGS[5], L=65536))):
            lsets = []
            for i in range(2):
                lx = make_layer(lw, layer=i)
                lsets.append(tuple(torch.from_numpy(b.view(np.int16)).to(dev).view(torch.bfloat16)
                                   for b in (lx.q_obs, lx.K, lx.V)))
            ln = ck.out_len(lw.L, lw.w, lw.c, lw.budget)
            lo = [torch.empty((lw.Hkv, ln, lw.d), dtype=torch.bfloat16, device=dev) for _ in range(2)]
            lo.append(torch.empty((lw.Hkv, ln), dtype=torch.int32, device=dev))
            cnt = [0]

            def long_layer():
                q, K, V = lsets[cnt[0] % 2]
                cnt[0] += 1
                st = lib.chunkkv_compress_layer(q.data_ptr(), K.data_ptr(), V.data_ptr(), lw.L, lw.Hq, lw.Hkv, lw.d, lw.w,
                                                lw.c, lw.budget, None, lo[0].data_ptr(), lo[1].data_ptr(),
                                                lo[2].data_ptr(), stream.cuda_stream)
                if st != 0:
                    raise ck.ChunkKVError(st, "chunkkv_compress_layer (long context)")

            with torch.cuda.stream(stream):
                us = time_calls(long_layer, n=20)
            if ck.device_status() != 0:
                raise RuntimeError("a kernel reported an abandoned wait")
            lb = layer_bytes(lw, ln)["layer"]
            R = lw.w * lw.Hq // lw.Hkv
            flops = 2.0 * R * lw.L * lw.d * lw.Hkv
            exps = float(R) * lw.L * lw.Hkv
            clock_max_mhz = clocks.get("sm_max_mhz")
            sfu_floor_us = exps / (16.0 * sm_count * clock_max_mhz * 1e6) * 1e6 if clock_max_mhz else None
            long_rows[name] = {
                "Hq": lw.Hq, "Hkv": lw.Hkv, "L": lw.L, "w": lw.w, "c": lw.c, "budget": lw.budget, "score_rows_per_kv_head": R,
                "us": us, "tokens_per_s": lw.L / (us * 1e-6), "algorithmic_bytes": lb,
                "GB/s": lb / (us * 1e-6) / 1e9, "frac_of_measured_hbm_peak": lb / (us * 1e-6) / 1e9 / peak,
                "bf16_TFLOP/s": flops / (us * 1e-6) / 1e12,
                "frac_of_sustained_bf16_peak": flops / (us * 1e-6) / 1e12 / tf_peak, "bf16_peak_source": tf_src,
                "exponentials": exps, "special_function_floor_us": sfu_floor_us,
                "note": "chunkkv_compress_layer, one layer at a time on all SMs, two K/V sets alternating (each > L2); "
                        "floor = exponentials / (16 per clock per SM at the maximum SM clock)"}
            del lsets, lo
        extra_roof["long_context_layers"] = long_rows

    # ---- end to end: pinned host buffers in, host buffers out, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        pin = []
        for x in hosts:
            pin.append([torch.from_numpy(b.view(np.int16)).view(torch.bfloat16).pin_memory()
                        for b in (x.q_obs, x.K, x.V)])
        h_out = [torch.empty((wl.Hkv, n_max, wl.d), dtype=torch.bfloat16).pin_memory() for _ in range(2)]
        h_out.append(torch.empty((wl.Hkv, n_max), dtype=torch.int32).pin_memory())

        def step_e2e():
            for i in range(LAYERS_PER_STEP):
                q, K, V = sets[i % NSETS][0]
                oK, oV, oI = lane_outs[0]
                hq, hK, hV = pin[i % NSETS]
                st = lib.chunkkv_compress_layer_host(
                    hq.data_ptr(), hK.data_ptr(), hV.data_ptr(), wl.L, wl.Hq, wl.Hkv, wl.d, wl.w, wl.c,
                    wl.budget, q.data_ptr(), K.data_ptr(), V.data_ptr(), oK.data_ptr(), oV.data_ptr(),
                    oI.data_ptr(), h_out[0].data_ptr(), h_out[1].data_ptr(), h_out[2].data_ptr(), stream.cuda_stream)
                if st != 0:
                    raise ck.ChunkKVError(st, "chunkkv_compress_layer_host")

        e2e_steps = max(1, min(args.steps, 3))
        timed(step_e2e, 1)
        ms_e2e = timed(step_e2e, e2e_steps)
        e2e_val, _ = job_throughput(e2e_steps * LAYERS_PER_STEP * wl.L, ms_e2e, dev)
        h2d = LAYERS_PER_STEP * (2 * wl.Hkv * wl.L * wl.d * 2 + wl.Hq * wl.w * wl.d * 2)
        d2h = LAYERS_PER_STEP * (2 * wl.Hkv * n_max * wl.d * 2 + wl.Hkv * n_max * 4)
        e2e = {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "steps": e2e_steps}
    if ck.device_status(stream) != 0 or any(ln.status() != 0 for ln in lanes):
        raise RuntimeError("a kernel reported an abandoned wait")

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = time_oracle(wl, hosts[0], budget_s=12.0)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "Hq": wl.Hq, "Hkv": wl.Hkv, "d": wl.d, "L": wl.L, "w": wl.w,
                       "c": wl.c, "budget": wl.budget, "layers_per_step": LAYERS_PER_STEP,
                       "lanes": S,
                       "mode": args.mode if S > 1 else "single",
                       "launch": f"one CUDA graph per step: 32 layer calls ({'chunkkv_pipe_layer' if piped else 'chunkkv_compress_layer_lane'}), {S} in flight "
                                 f"on {S} streams with {lane_ctas} CTAs each" if S > 1 else
                                 "one CUDA graph per step (32 chunkkv_compress_layer calls captured)",
                       "l2": f"layers cycle over {NSETS} distinct K/V sets of "
                             f"{2 * wl.Hkv * wl.L * wl.d * 2 / 1e6:.0f} MB each (> L2)"},
            "us_per_layer": ms_layer * 1e3,
            "eager": {"value": LAYERS_PER_STEP * wl.L * world / (ms_eager * 1e-3), "unit": UNIT,
                      "us_per_layer": ms_eager / LAYERS_PER_STEP * 1e3,
                      "note": "same step, 32 direct C-ABI calls, no graph"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": args.steps * LAYERS_PER_STEP * (launches_per_layer if fused else 5),
            "roofline": roofline, "roofline_more": extra_roof, "per_kernel": per_kernel,
            "cpu_baseline": cpu_baseline,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    from workloads import CONFIGS
    wl = CONFIGS[args.config]
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
