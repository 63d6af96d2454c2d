#!/usr/bin/env python
"""Benchmark of ChunkKV layer compression on B200 (one process per GPU).

Metric: prefix tokens compressed per second per layer, on the Llama-3-8B 32K KV shape
(Hq 32, Hkv 8, d 128, L 32768, w 32, c 10, budget 3276), seeded synthetic bf16 tensors.

A step compresses the 32 layers of one 32K-token sequence (score -> chunk-sum -> top-k -> gather
per layer). Every layer of the step has its own seeded q / K / V in HBM (32 x 134 MB), so no layer
finds another layer's keys in L2. `value` times the step as ONE chunkkv_compress_model call (the
persistent kernel: scoring of a layer overlaps selecting and gathering the one before), captured
in a CUDA graph and replayed; `eager` is the same call without a graph;
`roofline_more.single_layer` runs the same 32 layers as 32 chunkkv_compress_layer calls;
`roofline_more.shared_inputs` repeats the headline with the 32 layers pointing at only 4 distinct
K/V sets (what an L2-friendly input rotation would measure - for comparison only); `e2e` goes
through chunkkv_compress_layer_host with pinned host buffers, copies inside the timed region.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
  python bench.py --profile-case {layer,model,reuse,token,cfg4} [--iters n]   (a few calls, for ncu)
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
LAYERS_PER_STEP = 32
SHARED_SETS = 4
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
# DRAM bytes per layer of the persistent kernel, from the ncu capture summarised under profiles/ (4 layers, cfg2)
NCU_DRAM_BYTES_PER_LAYER = 338.2e6 / 4
NCU_TRAFFIC_WORKLOAD = "cfg2_llama3_8b_32k"
FALLBACK_BF16_SUSTAINED_TFLOPS = 1400.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=("ours", "reference"), default="ours")
    ap.add_argument("--config", type=int, default=2, help="workload table entry (2 = headline)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extra", action="store_true",
                    help="skip the secondary rows (long contexts, batched workload, token-level layers, sustained loop)")
    ap.add_argument("--profile-case", choices=("layer", "model", "reuse", "token", "cfg4"), default=None,
                    help="run a few calls of one case and exit (for use under a profiler)")
    ap.add_argument("--iters", type=int, default=3, help="calls of --profile-case")
    ap.add_argument("--layers", type=int, default=4, help="layers of --profile-case model")
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
def to_dev(bits, dev):
    return torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)


def make_layers(wl, n, dev, seq=0, workers=8):
    """n distinct seeded layers of a workload on the device (generated on host threads)."""
    from concurrent.futures import ThreadPoolExecutor
    from workloads import make_layer
    out = [None] * n
    with ThreadPoolExecutor(max_workers=workers) as ex:
        for i, x in enumerate(ex.map(lambda i: make_layer(wl, layer=i, seq=seq), range(n))):
            out[i] = (to_dev(x.q_obs, dev), to_dev(x.K, dev), to_dev(x.V, dev))
    return out


def alloc_outs(ck, wl, n, dev, c=None):
    n_max = ck.out_len(wl.L, wl.w, wl.c if c is None else c, wl.budget)
    return [(torch.empty((wl.Hkv, n_max, wl.d), dtype=torch.bfloat16, device=dev),
             torch.empty((wl.Hkv, n_max, wl.d), dtype=torch.bfloat16, device=dev),
             torch.empty((wl.Hkv, n_max), dtype=torch.int32, device=dev)) for _ in range(n)]


class ModelCall:
    """Marshalled arguments of one chunkkv_compress_model call (built once, issued many times)."""

    def __init__(self, ck, wl, layers, outs, reuse_depth, L=None):
        import ctypes
        self.ck, self.wl, self.n, self.reuse = ck, wl, len(layers), reuse_depth
        self.L = wl.L if L is None else L
        arr = ctypes.c_void_p * self.n
        self.q = arr(*[None if (i % reuse_depth) else t[0].data_ptr() for i, t in enumerate(layers)])
        self.K = arr(*[t[1].data_ptr() for t in layers])
        self.V = arr(*[t[2].data_ptr() for t in layers])
        self.oK = arr(*[o[0].data_ptr() for o in outs])
        self.oV = arr(*[o[1].data_ptr() for o in outs])
        self.oI = arr(*[o[2].data_ptr() for o in outs])
        self.keep = (layers, outs)
        need = int(ck.lib.chunkkv_model_workspace_bytes(self.n, self.L, wl.Hq, wl.Hkv, wl.d, wl.w, wl.c, wl.budget,
                                                        reuse_depth))
        self.workspace_bytes = need

    def __call__(self, stream):
        wl = self.wl
        st = self.ck.lib.chunkkv_compress_model(self.n, self.q, self.K, self.V, self.L, wl.Hq, wl.Hkv, wl.d, wl.w, wl.c,
                                                wl.budget, self.reuse, self.oK, self.oV, self.oI, stream.cuda_stream)
        if st != 0:
            raise self.ck.ChunkKVError(st, "chunkkv_compress_model")


def run_ours(args, wl):
    import torch.distributed as dist

    from paper_2502_00299_b200 import build as _build
    _build.build()
    import paper_2502_00299_b200 as ck
    from paper_2502_00299_b200 import binding as ckb
    from paper_2502_00299_b200.sharding import job_throughput, max_over_ranks
    from workloads import CONFIGS, iter_layers, make_layer, ragged_lengths, scaled

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
    NL = LAYERS_PER_STEP
    n_max = ck.out_len(wl.L, wl.w, wl.c, wl.budget)
    nbytes = layer_bytes(wl, n_max)
    peak, peak_src = measured_hbm_peak()
    stream = torch.cuda.Stream(device=dev)
    extra = not args.no_extra and rank == 0

    # ---- inputs: every layer of the step has its own q / K / V (rank r takes sequence r)
    layers = make_layers(wl, NL, dev, seq=rank)
    outs = alloc_outs(ck, wl, NL, dev)
    shared = [layers[i % SHARED_SETS] for i in range(NL)]            # 4 K/V sets standing in for 32 layers
    model = ModelCall(ck, wl, layers, outs, 1)
    model_shared = ModelCall(ck, wl, shared, outs, 1)
    model_reuse2 = ModelCall(ck, wl, layers, outs, 2)
    # the library allocates nothing: one scratch buffer that covers every shape timed below, handed
    # over once, before anything is captured in a graph
    need = max(model.workspace_bytes, model_reuse2.workspace_bytes,
               ck.workspace_bytes(wl.L, wl.Hq, wl.Hkv, wl.d, wl.w, wl.c),
               ck.workspace_bytes(wl.L, wl.Hq, wl.Hkv, wl.d, wl.w, 1))
    long_cfgs = (("cfg4_128k", CONFIGS[4]), ("cfg5_longest_64k", scaled(CONFIGS[5], L=65536)))
    lens5 = ragged_lengths(CONFIGS[5])
    if extra:
        for _, lw in long_cfgs:
            need = max(need, ck.workspace_bytes(lw.L, lw.Hq, lw.Hkv, lw.d, lw.w, lw.c))
        w5 = CONFIGS[5]
        for L5 in lens5:
            need = max(need, int(lib.chunkkv_model_workspace_bytes(w5.n_layers, L5, w5.Hq, w5.Hkv, w5.d, w5.w, w5.c,
                                                                   w5.budget, w5.reuse_depth)),
                       ck.workspace_bytes(L5, w5.Hq, w5.Hkv, w5.d, w5.w, w5.c))
    ckb._ensure_bytes(int(need))

    def layer_call(i, reuse=False, c=None, o=None, src=None):
        q, K, V = (layers if src is None else src)[i]
        oK, oV, oI = (outs if o is None else o)[i]
        st = lib.chunkkv_compress_layer(None if reuse else q.data_ptr(), K.data_ptr(), V.data_ptr(), wl.L, wl.Hq, wl.Hkv,
                                        wl.d, wl.w, wl.c if c is None else c, wl.budget, oI.data_ptr() if reuse else None,
                                        oK.data_ptr(), oV.data_ptr(), oI.data_ptr(), stream.cuda_stream)
        if st != 0:
            raise ck.ChunkKVError(st, "chunkkv_compress_layer")

    def step_single():
        for i in range(NL):
            layer_call(i)

    def step_reuse():
        for i in range(NL):
            layer_call(i, reuse=True)

    def capture(fn):
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr, stream=stream):
            fn()
        return gr

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

    def check_status():
        if ck.device_status(stream) != 0:
            raise RuntimeError("a kernel reported an abandoned wait")

    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
            model(stream)
            step_single()
            step_reuse()
    torch.cuda.synchronize()
    check_status()
    g_model = capture(lambda: model(stream))
    g_shared = capture(lambda: model_shared(stream))
    g_reuse2 = capture(lambda: model_reuse2(stream))
    g_single = capture(step_single)
    g_reuse = capture(step_reuse)
    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
            for g in (g_model, g_shared, g_reuse2, g_single, g_reuse):
                g.replay()
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        gpu_id = str(local_rank)

    # ---- headline: one chunkkv_compress_model call per step, as a replayed graph
    sampler = ClockSampler(gpu_id)
    sampler.start()
    ms_total = timed(g_model.replay, args.steps)
    clocks = sampler.stop()
    value, ms_max = job_throughput(args.steps * NL * wl.L, ms_total, dev)
    ms_per_step = ms_max / args.steps
    us_layer = ms_per_step / NL * 1e3

    few = max(3, min(args.steps, 100))
    us_eager = max_over_ranks(timed(lambda: model(stream), few), dev) / few / NL * 1e3
    us_shared = max_over_ranks(timed(g_shared.replay, few), dev) / few / NL * 1e3
    us_single = max_over_ranks(timed(g_single.replay, few), dev) / few / NL * 1e3
    us_reuse = max_over_ranks(timed(g_reuse.replay, few), dev) / few / NL * 1e3
    us_reuse2_model = max_over_ranks(timed(g_reuse2.replay, few), dev) / few * 1e3      # per 32-layer model
    check_status()

    def frac_row(nb, us, **kw):
        gbs = nb / (us * 1e-6) / 1e9
        row = {"algorithmic_bytes": nb, "us": us, "GB/s": gbs, "frac_of_measured_peak": gbs / peak,
               "frac_of_8TBps": gbs / NOMINAL_HBM_GBS}
        row.update(kw)
        return row

    # per-kernel durations of the call-by-call path (CUDA events around every launch, one layer at a time)
    ck.profile_enable(True)
    timed(step_single, 3)
    ms_slot, n_slot = ck.profile_read()
    ck.profile_enable(False)
    names = ("layer_or_score", "finalize", "select", "gather")
    per_kernel = {n: {"launches": c, "avg_us": (m / c * 1e3) if c else None, "total_ms": m}
                  for n, m, c in zip(names, ms_slot, n_slot)}
    iso_us = per_kernel["layer_or_score"]["avg_us"] or float("nan")

    achieved = nbytes["layer"] * NL / (ms_per_step * 1e-3) / 1e9
    roofline = {
        "kernel": "model_kernel<10>: the persistent kernel behind chunkkv_compress_model - 32 layers per launch; "
                  "scoring (TMA + tcgen05), chunk sums in tensor memory, top-k on selector CTAs, row copies by bulk copy",
        "bound": "hbm", "achieved": achieved, "peak": peak, "peak_source": peak_src, "unit": "GB/s",
        "frac": achieved / peak, "frac_of_8TBps": achieved / NOMINAL_HBM_GBS,
        "traffic": NCU_DRAM_BYTES_PER_LAYER * NL if wl.name == NCU_TRAFFIC_WORKLOAD else None,
        "traffic_source": "ncu dram__bytes_read.sum + dram__bytes_write.sum of one 4-layer launch of the same kernel on this "
                          "workload (profiles/model_kernel_cfg2_4layers_ncu.txt: 338.2 MB), per layer x the 32 layers of a "
                          "launch: every layer streams its own K once, so the traffic grows with the layers; the 32-layer "
                          "launch itself is too large for a counter capture",
        "algorithmic_bytes_per_launch": nbytes["layer"] * NL, "avg_launch_us": ms_per_step * 1e3,
        "launches_per_step": 1, "layers_per_launch": NL,
        "isolated_launch_us": iso_us,
        "isolated_frac": nbytes["layer"] / (iso_us * 1e-6) / 1e9 / peak,
        "note": "avg_launch_us = CUDA-event time of the timed region / launches in it (one launch per step, nothing else "
                "in the region); algorithmic bytes = 32 x (K once + q + K/V rows read and written); isolated_* = the "
                "one-layer kernel of chunkkv_compress_layer with events around every launch, same distinct inputs"}
    extra_roof = {
        "model_call": frac_row(nbytes["layer"], us_layer, note="headline: per layer inside one 32-layer chunkkv_compress_model call"),
        "single_layer": frac_row(nbytes["layer"], us_single,
                                 note="32 chunkkv_compress_layer calls back to back (one kernel per layer, each on all SMs), as a graph"),
        "shared_inputs": frac_row(nbytes["layer"], us_shared,
                                  note=f"headline call with the 32 layers pointing at {SHARED_SETS} K/V sets (L2 can serve repeats): "
                                       "comparison only, not a roofline number"),
        "reuse_layer": frac_row(nbytes["gather"], us_reuse, note="gather-only layers (index reuse), one launch each"),
    }

    # ---- 32 layers with reuse depth 2 (the paper's index-reuse setting), against its speed-up model
    t_c, t_sel = us_layer, us_reuse
    n_r = 2
    modelled = NL * t_c / (NL / n_r * t_c + (NL - NL / n_r) * t_sel)
    extra_roof["cfg3_model"] = {
        "layers": NL, "reuse_depth": n_r, "us_per_model": us_reuse2_model, "us_per_model_all_layers_computed": us_layer * NL,
        "measured_speedup": us_layer * NL / us_reuse2_model, "modelled_speedup": modelled,
        "T_compress_us": t_c, "T_select_us": t_sel,
        "note": "one chunkkv_compress_model call, 16 computed + 16 reusing layers, distinct K/V per layer; modelled = "
                "N T_c / (N/N_r T_c + (N - N/N_r) T_sel) with T_c = headline per-layer time, T_sel = gather-only layer time"}

    def time_calls(fn, n=30):
        for _ in range(3):
            fn()
        return timed(lambda: [fn() for _ in range(n)], 1) / n * 1e3      # us per call

    if extra:
        # adjacent computed layers of the correlated 32-layer workload: how much their kept sets overlap
        w3 = CONFIGS[3]
        l3 = []
        for x in iter_layers(w3, 3):
            l3.append((to_dev(x.q_obs, dev), to_dev(x.K, dev), to_dev(x.V, dev)))
        with torch.cuda.stream(stream):
            o3 = ck.compress_model(l3, w3.Hq, w3.w, w3.c, w3.budget, n_reuse=2, stream=stream)
            ratio, _ = ck.jaccard(o3[0][2], o3[2][2], stream=stream)
            us_jac = time_calls(lambda: ck.jaccard(o3[0][2], o3[2][2], stream=stream))
        torch.cuda.synchronize()
        extra_roof["cfg3_model"]["adjacent_computed_layer_jaccard"] = {
            "mean": float(ratio.mean()), "min": float(ratio.min()), "max": float(ratio.max()),
            "note": "chunkkv_jaccard of the kept indices of layers 0 and 2 of the correlated workload (rho 0.8), per KV head"}
        extra_roof["jaccard"] = {"us": us_jac, "note": "chunkkv_jaccard on two [8, 3272] index matrices (latency-bound)"}
        del l3, o3

        # ---- sustained: the headline graph for at least a second, with the clocks it ran at
        reps = int(max(1.0, 1.2e3 / max(ms_per_step, 1e-3)))
        s2 = ClockSampler(gpu_id)
        s2.start()
        ms_sus = timed(g_model.replay, reps)
        c2 = s2.stop()
        extra_roof["sustained"] = frac_row(nbytes["layer"], ms_sus / reps / NL * 1e3, seconds=ms_sus * 1e-3, steps=reps,
                                           clocks=c2, note="headline step replayed for more than a second")

        # ---- token-level layers (c = 1) through chunkkv_compress_layer
        o1 = alloc_outs(ck, wl, 2, dev, c=1)
        cnt = [0]

        def token_level_layer():
            i = cnt[0] % NL
            cnt[0] += 1
            layer_call(i, c=1, o=[o1[i % 2]] * NL)

        with torch.cuda.stream(stream):
            us_token_eager = time_calls(token_level_layer)
        cnt[0] = 0
        g_token = capture(lambda: [token_level_layer() for _ in range(NL)])
        timed(g_token.replay, 3)
        us_token = timed(g_token.replay, few) / few / NL * 1e3
        b1 = layer_bytes(wl, ck.out_len(wl.L, wl.w, 1, wl.budget))["layer"]
        extra_roof["token_level_layer"] = frac_row(
            b1, us_token, c=1, us_eager=us_token_eager,
            note="32 chunkkv_compress_layer calls with c = 1 on the 32 distinct layers, back to back, as a graph (the way "
                 "single_layer is timed); us_eager = the same calls issued directly")
        del o1, g_token

        # ---- the adapters either side of the path and Algorithm 1's budget rule, on the same layers
        #      (one call at a time, issued directly; the bindings' output allocations are outside the loop)
        ad = {}
        oA = alloc_outs(ck, wl, 1, dev)[0]
        qi, Ki, Vi = layers[0]
        tmK = Ki.permute(1, 0, 2).contiguous()                  # a token-major cache [L, Hkv, d]
        tmV = Vi.permute(1, 0, 2).contiguous()
        vK, vV = tmK.permute(1, 0, 2), tmV.permute(1, 0, 2)

        def strided_layer():
            ck.compress_layer_strided(qi, vK, vV, wl.Hq, wl.w, wl.c, wl.budget, out_K=oA[0], out_V=oA[1], out_idx=oA[2],
                                      stream=stream)

        page = 16
        n_blk = (n_max + page - 1) // page
        table = torch.randperm(n_blk, device=dev).to(torch.int32)
        cK = torch.empty((n_blk, page, wl.Hkv, wl.d), dtype=torch.bfloat16, device=dev)
        cV = torch.empty_like(cK)

        def paged_layer():
            ck.compress_layer_paged(qi, Ki, Vi, wl.Hq, wl.w, wl.c, wl.budget, table, cK, cV, out_idx=oA[2], stream=stream)

        n1 = ck.out_len_alg1(wl.L, wl.w, wl.c, wl.budget)
        o1a = (torch.empty((wl.Hkv, n1, wl.d), dtype=torch.bfloat16, device=dev),
               torch.empty((wl.Hkv, n1, wl.d), dtype=torch.bfloat16, device=dev),
               torch.empty((wl.Hkv, n1), dtype=torch.int32, device=dev))

        def alg1_layer():
            ck.compress_layer_alg1(qi, Ki, Vi, wl.Hq, wl.w, wl.c, wl.budget, out_K=o1a[0], out_V=o1a[1], out_idx=o1a[2],
                                   stream=stream)

        T = 4 * wl.w
        row = (wl.Hq + 2 * wl.Hkv) * wl.d
        qkv = torch.randn((T, row), device=dev).to(torch.bfloat16)
        ang = torch.rand((wl.w, wl.d // 2), device=dev) * 6.28
        cos_r, sin_r = torch.cos(ang), torch.sin(ang)

        def window_q():
            ck.window_queries(qkv, wl.Hq, wl.Hkv, wl.d, wl.w, cos_r, sin_r, stream=stream)

        with torch.cuda.stream(stream):
            for name, fn, nb in (("compress_layer_strided", strided_layer, nbytes["layer"]),
                                 ("compress_layer_paged", paged_layer, nbytes["layer"]),
                                 ("compress_layer_alg1", alg1_layer, nbytes["layer"]),
                                 ("window_queries", window_q, None)):
                us_a = time_calls(fn)
                ad[name] = {"us": us_a} if nb is None else frac_row(nb, us_a)
            tm8 = []
            for q8, K8, V8 in layers[:8]:
                tm8.append((q8, K8.permute(1, 0, 2).contiguous().permute(1, 0, 2), V8.permute(1, 0, 2).contiguous().permute(1, 0, 2)))
            us_m = time_calls(lambda: ck.compress_model_strided(tm8, wl.Hq, wl.w, wl.c, wl.budget, n_reuse=1, outs=outs[:8],
                                                                stream=stream), n=10) / 8
            ad["compress_model_strided"] = frac_row(nbytes["layer"], us_m, layers_per_call=8)
            del tm8
            tabs8 = [torch.randperm(n_blk, device=dev).to(torch.int32) for _ in range(8)]
            caches8 = [(torch.empty_like(cK), torch.empty_like(cV)) for _ in range(8)]
            idx8 = [o[2] for o in outs[:8]]
            us_p = time_calls(lambda: ck.compress_model_paged(layers[:8], wl.Hq, wl.w, wl.c, wl.budget, tabs8, caches8, n_reuse=1,
                                                              stream=stream, out_idx=idx8), n=10) / 8
            ad["compress_model_paged"] = frac_row(nbytes["layer"], us_p, layers_per_call=8)
            del caches8
        ad["note"] = ("cfg2 layer: keys and values read from a token-major cache [L, Hkv, d]; kept rows written to a paged cache "
                      "(16 tokens per page, shuffled block table); Algorithm 1's budget rule; the last w rows of a fused QKV "
                      "activation rotated into q_obs (includes the binding's output allocation); compress_model_strided / _paged: 8 layers "
                      "per call (token-major inputs / paged outputs), us per layer")
        extra_roof["adapters"] = ad
        del tmK, tmV, cK, cV, o1a, qkv
        check_status()
        check_status()

    del g_model, g_shared, g_reuse2, g_single, g_reuse, model, model_shared, model_reuse2
    hosts0 = None
    if not args.no_e2e or (rank == 0 and world == 1 and not args.no_cpu_baseline):
        hosts0 = make_layer(wl, layer=0, seq=rank)

    if extra:
        # ---- the long-context shapes (256 score rows per KV head: bound by exponentials and the tensor
        #      pipe rather than by HBM), one layer at a time on the whole GPU
        del layers, shared
        torch.cuda.empty_cache()
        tf_peak, tf_src = measured_bf16_sustained_tflops()
        sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
        long_rows = {}
        for name, lw in long_cfgs:
            ll = make_layers(lw, 2, dev)
            lo = alloc_outs(ck, lw, 1, dev)[0]
            cnt = [0]

            def long_layer():
                q, K, V = ll[cnt[0] % 2]
                cnt[0] += 1
                st = lib.chunkkv_compress_layer(q.data_ptr(), K.data_ptr(), V.data_ptr(), lw.L, lw.Hq, lw.Hkv, lw.d, lw.w,
                                                lw.c, lw.budget, None, lo[0].data_ptr(), lo[1].data_ptr(),
                                                lo[2].data_ptr(), stream.cuda_stream)
                if st != 0:
                    raise ck.ChunkKVError(st, "chunkkv_compress_layer (long context)")

            with torch.cuda.stream(stream):
                us = time_calls(long_layer, n=20)
            check_status()
            lb = layer_bytes(lw, ck.out_len(lw.L, lw.w, lw.c, lw.budget))["layer"]
            R = lw.w * lw.Hq // lw.Hkv
            flops = 2.0 * R * lw.L * lw.d * lw.Hkv
            exps = float(R) * lw.L * lw.Hkv
            mhz = clocks.get("sm_max_mhz")
            row = frac_row(lb, us, Hq=lw.Hq, Hkv=lw.Hkv, L=lw.L, w=lw.w, c=lw.c, budget=lw.budget, score_rows_per_kv_head=R,
                           tokens_per_s=lw.L / (us * 1e-6))
            row.update({"bf16_TFLOP/s": flops / (us * 1e-6) / 1e12,
                        "frac_of_sustained_bf16_peak": flops / (us * 1e-6) / 1e12 / tf_peak, "bf16_peak_source": tf_src,
                        "exponentials": exps,
                        "special_function_floor_us": exps / (16.0 * sm_count * mhz * 1e6) * 1e6 if mhz else None,
                        "note": "chunkkv_compress_layer, one layer at a time on all SMs, two K/V sets alternating (each > L2); "
                                "floor = exponentials / (16 per clock per SM at the maximum SM clock)"})
            long_rows[name] = row
            del ll, lo
        extra_roof["long_context_layers"] = long_rows

        # ---- the batched serving workload as configured: 8 ragged sequences x 80 layers, reuse depth 3.
        #      Each sequence cycles a ring of 6 layer buffers at distinct addresses (two seeded layers,
        #      replicated on the device); one chunkkv_compress_model call per sequence.
        w5 = CONFIGS[5]
        n5 = ck.out_len(w5.L, w5.w, w5.c, w5.budget)
        outs5 = [(torch.empty((w5.Hkv, n5, w5.d), dtype=torch.bfloat16, device=dev),
                  torch.empty((w5.Hkv, n5, w5.d), dtype=torch.bfloat16, device=dev),
                  torch.empty((w5.Hkv, n5), dtype=torch.int32, device=dev)) for _ in range(w5.n_layers)]
        calls5 = []
        for b, L5 in enumerate(lens5):
            wb = scaled(w5, L=L5)
            base = make_layers(wb, 2, dev, seq=b)
            ring = [base[i % 2] if i < 2 else tuple(t.clone() for t in base[i % 2]) for i in range(6)]
            calls5.append(ModelCall(ck, wb, [ring[l % 6] for l in range(w5.n_layers)], outs5, w5.reuse_depth, L=L5))

        def batch_step():
            for mc in calls5:
                mc(stream)

        with torch.cuda.stream(stream):
            for _ in range(2):
                batch_step()
        torch.cuda.synchronize()
        check_status()
        ms5 = timed(batch_step, 3) / 3
        n_comp = (w5.n_layers + w5.reuse_depth - 1) // w5.reuse_depth
        bytes5 = 0
        for L5 in lens5:
            lb5 = layer_bytes(scaled(w5, L=L5), n5)
            bytes5 += n_comp * lb5["layer"] + (w5.n_layers - n_comp) * lb5["gather"]
        extra_roof["cfg5_batch"] = {
            "sequences": len(lens5), "lengths": list(lens5), "layers": w5.n_layers, "reuse_depth": w5.reuse_depth,
            "ms_per_batch": ms5, "tokens_per_s_per_layer": sum(lens5) * w5.n_layers / (ms5 * 1e-3),
            "algorithmic_bytes": bytes5, "GB/s": bytes5 / (ms5 * 1e-3) / 1e9,
            "frac_of_measured_peak": bytes5 / (ms5 * 1e-3) / 1e9 / peak,
            "note": "8 chunkkv_compress_model calls (one per sequence, 27 computed + 53 reusing layers each), sequences one "
                    "after another; sequences too long for the persistent kernel's tensor-memory budget run layer by layer"}
        del calls5, outs5
        torch.cuda.empty_cache()

    # ---- end to end: pinned host buffers in, host buffers out, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        pin = [torch.from_numpy(b.view(np.int16)).view(torch.bfloat16).pin_memory()
               for b in (hosts0.q_obs, hosts0.K, hosts0.V)]
        stage = [torch.empty_like(t, device=dev) for t in pin]
        oK, oV, oI = outs[0]
        h_out = [torch.empty((wl.Hkv, n_max, wl.d), dtype=torch.bfloat16).pin_memory() for _ in range(2)]
        h_out.append(torch.empty((wl.Hkv, n_max), dtype=torch.int32).pin_memory())
        e2e_layers = 8

        def step_e2e():
            for _ in range(e2e_layers):
                st = lib.chunkkv_compress_layer_host(
                    pin[0].data_ptr(), pin[1].data_ptr(), pin[2].data_ptr(), wl.L, wl.Hq, wl.Hkv, wl.d, wl.w, wl.c,
                    wl.budget, stage[0].data_ptr(), stage[1].data_ptr(), stage[2].data_ptr(), oK.data_ptr(), oV.data_ptr(),
                    oI.data_ptr(), h_out[0].data_ptr(), h_out[1].data_ptr(), h_out[2].data_ptr(), stream.cuda_stream)
                if st != 0:
                    raise ck.ChunkKVError(st, "chunkkv_compress_layer_host")

        e2e_steps = 3
        timed(step_e2e, 1)
        ms_e2e = timed(step_e2e, e2e_steps)
        e2e_val, _ = job_throughput(e2e_steps * e2e_layers * wl.L, ms_e2e, dev)
        h2d = NL * (2 * wl.Hkv * wl.L * wl.d * 2 + wl.Hq * wl.w * wl.d * 2)
        d2h = NL * (2 * wl.Hkv * n_max * wl.d * 2 + wl.Hkv * n_max * 4)
        e2e = {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "note": f"chunkkv_compress_layer_host, {e2e_layers} layers per timed repetition x {e2e_steps}; bytes are per "
                       f"{NL}-layer step; bound by the host link"}
        check_status()

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = time_oracle(wl, hosts0, budget_s=12.0)
        cpu_baseline["single_thread"] = time_oracle_single_thread(wl, hosts0, budget_s=6.0)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "Hq": wl.Hq, "Hkv": wl.Hkv, "d": wl.d, "L": wl.L, "w": wl.w,
                       "c": wl.c, "budget": wl.budget, "layers_per_step": NL,
                       "launch": "one CUDA graph per step holding one chunkkv_compress_model call (32 computed layers, "
                                 "one persistent kernel launch)",
                       "l2": f"every layer of the step has its own seeded q / K / V: {NL} x "
                             f"{2 * wl.Hkv * wl.L * wl.d * 2 / 1e6:.0f} MB resident (> L2), none shared"},
            "us_per_layer": us_layer,
            "eager": {"value": NL * wl.L * world / (us_eager * NL * 1e-6), "unit": UNIT, "us_per_layer": us_eager,
                      "note": "same step, the C-ABI call issued directly, no graph"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": args.steps,
            "roofline": roofline, "roofline_more": extra_roof, "per_kernel": per_kernel,
            "cpu_baseline": cpu_baseline,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def time_oracle_single_thread(wl, x, budget_s: float):
    """The oracle on one thread: one KV head of one layer (scaled to a layer in the text only)."""
    from oracle import chunkkv_oracle as ora
    from threadpoolctl import threadpool_limits
    G = wl.Hq // wl.Hkv
    with threadpool_limits(limits=1):
        t0 = time.perf_counter()
        ora.compress_layer(x.q_obs[:G], x.K[:1], x.V[:1], G, 1, wl.w, wl.c, wl.budget)
        t1 = time.perf_counter() - t0
        n = int(max(1, min(20, round(budget_s / max(t1, 1e-3)))))
        t0 = time.perf_counter()
        for _ in range(n):
            ora.compress_layer(x.q_obs[:G], x.K[:1], x.V[:1], G, 1, wl.w, wl.c, wl.budget)
        dt = (time.perf_counter() - t0) / n
    return {"value": wl.L / (dt * wl.Hkv), "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{n} x one KV head of one {wl.name} layer on one thread, {dt * 1e3:.1f} ms per head; "
                      f"value = L / ({wl.Hkv} heads x that)"}


def run_profile_case(args):
    """A few calls of one case with little warm-up, for use under a profiler (ncu -k / -s / -c)."""
    import paper_2502_00299_b200 as ck
    from workloads import CONFIGS, scaled
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    case = args.profile_case
    wl = CONFIGS[4] if case == "cfg4" else CONFIGS[args.config]
    n = args.layers if case == "model" else 2
    layers = make_layers(wl, n, dev)
    c = 1 if case == "token" else wl.c
    outs = alloc_outs(ck, wl, n, dev, c=c)
    stream = torch.cuda.current_stream()
    times = []

    def run_once(i):
        if case == "model":
            ck.compress_model(layers, wl.Hq, wl.w, wl.c, wl.budget, n_reuse=1, outs=outs)
        else:
            q, K, V = layers[i % n]
            ck.compress_layer(q, K, V, wl.Hq, wl.w, c, wl.budget, reuse_idx=outs[i % n][2] if case == "reuse" else None,
                              out_K=outs[i % n][0], out_V=outs[i % n][1], out_idx=outs[i % n][2])

    if case == "reuse":
        ck.compress_layer(*layers[0], wl.Hq, wl.w, c, wl.budget, out_K=outs[0][0], out_V=outs[0][1], out_idx=outs[0][2])
        outs[1][2].copy_(outs[0][2])
    run_once(0)
    torch.cuda.synchronize()
    for it in range(args.iters):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        run_once(it)
        e1.record()
        times.append((e0, e1))
    torch.cuda.synchronize()
    assert ck.device_status() == 0
    print(case, wl.name, "us per call:", [round(a.elapsed_time(b) * 1e3, 1) for a, b in times], flush=True)


def spawn_ranks(args):
    """`python bench.py --gpus N` without a launcher: start N ranks of this script on this node."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "WARN")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd, env=env)


def main():
    args = parse_args()
    from workloads import CONFIGS
    wl = CONFIGS[args.config]
    if args.profile_case is not None:
        run_profile_case(args)
    elif args.impl == "reference":
        run_reference(args, wl)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
