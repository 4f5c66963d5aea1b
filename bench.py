#!/usr/bin/env python
"""Benchmark of the Virtual-Expert MoE-layer forward on B200.

One "step" is one pass of the whole hot path (router+gate, scan, permute, grouped
FFN GEMMs, combine, importance) over one batch of synthetic tokens.  The default
workload is the Switch-base-64-shaped layer (bf16, d_model 768, d_ff 3072, E 64,
top-1, K 16 resident slots, 2048 tokens with Zipf(1.1) expert popularity and
runs of 32 tokens sharing a preferred expert set).

    python bench.py --gpus 1 --steps 50 --warmup 10
    python bench.py --impl reference            # the CPU oracle on the host cores

Prints ONE JSON line.  With --gpus N > 1 (under torchrun) every rank runs an
independent replica on its own tokens ("replicas only": the path has no
exchange step), rank 0 prints the aggregate.
"""
from __future__ import annotations

import argparse
import gc
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2308_15030_b200 import inputs as I  # noqa: E402



def ncu_traffic(name):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of the grouped-GEMM kernel (mean of the GEMM-1
    and GEMM-2 launches of one step), as recorded beside the ncu summaries in profiles/ncu_traffic.json
    together with the commit the capture was taken at; None for workloads without a capture."""
    try:
        rec = json.load(open(os.path.join(ROOT, "profiles", "ncu_traffic.json"))).get(name)
    except (OSError, ValueError):
        return None, None
    if not rec:
        return None, None
    return float(rec["grouped_gemm_dram_bytes_per_launch"]), rec

METRIC = "moe_layer_tokens_per_s_at_budget_K"
UNIT = "tokens/s"
L2_BYTES = 126e6


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


def workload_string(cfg):
    return ("%s: %s d_model=%d d_ff=%d E=%d top%d K=%d resident T=%d tokens %s, zipf_s=%.1f "
            "runs of %d" % (cfg.name, "bf16" if cfg.dtype == I.BF16 else "fp32", cfg.d, cfg.f, cfg.E,
                            cfg.k, cfg.K, cfg.T, "SwiGLU" if cfg.act else "ReLU", cfg.zipf_s,
                            cfg.run_len))


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []
        self.t_begin = None      # wall-clock window of the timed regions (samples outside are dropped)

    def mark_begin(self):
        import datetime
        self.t_begin = datetime.datetime.now()

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        import datetime
        t_end = datetime.datetime.now()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [s.strip() for s in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f")
                if self.t_begin is not None and not (self.t_begin <= ts <= t_end):
                    continue
                f = f[1:]
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(mx)) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------- the CUDA arm
def algorithmic_bytes(cfg, touched):
    """Method's own traffic of one forward: resident weights that received >= 1 token,
    x in, out out, router matrix (implementation round trips of xp/h/y are excluded)."""
    return touched * cfg.nmat * cfg.d * cfg.f * cfg.nb + 2 * cfg.T * cfg.d * cfg.nb + cfg.E * cfg.d * cfg.nb


def gemm_algorithmic(cfg, touched):
    """Bytes and flops of the two grouped-GEMM launches of one forward: the touched
    slots' weights, the permuted tokens in and the expert outputs out; the hidden
    activations between the two GEMMs are an implementation round trip."""
    pairs = cfg.T * cfg.k
    nbytes = touched * cfg.nmat * cfg.d * cfg.f * cfg.nb + 2 * pairs * cfg.d * cfg.nb
    flops = 2.0 * pairs * cfg.d * cfg.f * cfg.nmat
    return nbytes, flops


def roofline_objects(cfg, touched, g_ms, ms_step, peaks):
    """`roofline` of the dominant kernel (the grouped GEMM: 2 launches per step) and the layer's own roofline."""
    g_bytes, g_flops = gemm_algorithmic(cfg, touched)
    # Tensor peak: kernels timed inside a long, power-capped step (>= 1 ms per step) are held against
    # the sustained cuBLAS figure, short ones against the burst figure.
    tc_kind = "sustained" if ms_step >= 1.0 else "burst"
    tc_peak = peaks["bf16_tflops_sustained"] if tc_kind == "sustained" else peaks["bf16_tflops"]
    t_hbm = g_bytes / (peaks["hbm_gbs"] * 1e9)
    t_tc = g_flops / (tc_peak * 1e12) if cfg.dtype == I.BF16 else 0.0
    # fp32 layers: the grouped GEMM runs on the tensor cores as three reduced-precision products per fp32 product:
    # bf16 pieces on tcgen05 (peak = the measured bf16 figure / 3), TF32 pieces in the warp-level mma kernels
    # (SWAPMOE_FP32_TC=0; peak = measured bf16 x the nominal TF32 : bf16 ratio, 1.1 : 2.25 PFLOP/s, / 3).
    fp32_mma = os.environ.get("SWAPMOE_FP32_TC") == "0"
    tf32x3_peak = peaks["bf16_tflops"] * ((1.1 / 2.25) if fp32_mma else 1.0) / 3.0
    if cfg.dtype != I.BF16 and t_hbm >= g_flops / (tf32x3_peak * 1e12):
        bound, peak, ach, unit = "hbm", peaks["hbm_gbs"], g_bytes / 2 / (g_ms * 1e-3) / 1e9, "GB/s"
    elif cfg.dtype != I.BF16:
        bound, peak, ach, unit = "tensor", tf32x3_peak, g_flops / 2 / (g_ms * 1e-3) / 1e12, "TFLOP/s"
    elif t_hbm >= t_tc:
        bound, peak, ach, unit = "hbm", peaks["hbm_gbs"], g_bytes / 2 / (g_ms * 1e-3) / 1e9, "GB/s"
    else:
        bound, peak, ach, unit = "tensor", tc_peak, g_flops / 2 / (g_ms * 1e-3) / 1e12, "TFLOP/s"
    layer_bytes = algorithmic_bytes(cfg, touched)
    layer_flops = 2.0 * cfg.T * cfg.d * cfg.E + g_flops
    t_roof = max(layer_bytes / (peaks["hbm_gbs"] * 1e9),
                 layer_flops / (tc_peak * 1e12) if cfg.dtype == I.BF16 else layer_flops / (tf32x3_peak * 1e12))
    traffic, traffic_rec = ncu_traffic(cfg.name)
    if cfg.dtype == I.BF16:
        kernel = "tc_gemm_kernel / tc_gemm_pair_kernel (grouped FFN GEMM on tcgen05, 2 launches per step: GEMM-1+act, GEMM-2)"
    elif fp32_mma:
        kernel = "gemm_tf32x3_kernel (split-TF32 warp-level mma, 2 launches per step)"
    else:
        kernel = "tc_gemm_f32_kernel (three products of bf16 pieces on tcgen05, 2 launches per step)"
    roof = {"bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak,
            "traffic": traffic, "traffic_source": traffic_rec, "peak_source": peaks["source"], "kernel": kernel,
            "algorithmic_bytes_per_launch": g_bytes / 2, "flops_per_launch": g_flops / 2,
            "avg_launch_ms": g_ms, "tensor_tflops": g_flops / 2 / (g_ms * 1e-3) / 1e12,
            "tensor_peak_kind": (tc_kind if cfg.dtype == I.BF16 else
                                 ("bf16 burst x 1.1/2.25 / 3 (TF32 x3)" if fp32_mma else "bf16 burst / 3 (bf16 pieces x3)"))
                                if bound == "tensor" else None,
            "frac_of_burst_tensor_peak": (ach / peaks["bf16_tflops"]) if bound == "tensor" else None}
    layer = {"t_roof_us": t_roof * 1e6, "frac": t_roof * 1e3 / ms_step,
             "algorithmic_bytes": layer_bytes, "flops": layer_flops}
    return roof, layer


MIN_REGION_MS = 250.0      # the timed loop is repeated until it covers at least this much device time


def measure_layer(cfg, steps, warmup, *, rank=0, world=1, local=0, no_graph=False, want_e2e=True,
                  sampler=None, barrier=None, min_region_ms=MIN_REGION_MS):
    """Times `steps` forwards of one layer configuration (device-resident inputs), a stage-event pass,
    a warm-cache loop and, if asked, the end-to-end host-buffer path.  Returns a dict of raw figures."""
    import torch
    from paper_2308_15030_b200 import binding

    tdt = torch.bfloat16 if cfg.dtype == I.BF16 else torch.float32
    if barrier is None:
        barrier = torch.cuda.synchronize

    def dev(a):
        a = np.ascontiguousarray(a, dtype=np.float32)
        if cfg.dtype == I.BF16:
            return torch.from_numpy(I.bf16_bits(a).view(np.int16)).view(torch.bfloat16).cuda()
        return torch.from_numpy(a).cuda()

    Wr = I.make_router(cfg)
    enorm = I.make_enorm(cfg)
    # every rank draws its own tokens (replicas on different batches)
    x_host = I.make_tokens(cfg, Wr, seed=cfg.seed + 1000 * rank)
    d_Wr = dev(Wr)
    weight_bytes = cfg.K * cfg.nmat * cfg.d * cfg.f * cfg.nb
    copies = max(1, int(np.ceil(4 * L2_BYTES / weight_bytes)))   # rotation spans > 4x L2
    stream = torch.cuda.Stream()

    # Resident set chosen the product's own way: one pass with an arbitrary set to
    # collect Eq. (1) importance, then the top-K experts become resident.
    d_x = [dev(x_host) for _ in range(copies)]
    d_out = [torch.empty((cfg.T, cfg.d), dtype=tdt, device="cuda") for _ in range(copies)]
    with torch.cuda.stream(stream):
        first = list(range(cfg.K))
        a_in, a_out = I.build_arena(cfg, first)
        arenas = [(dev(a_in), dev(a_out))]
        layers = [binding.Layer(cfg.E, cfg.d, cfg.f, cfg.k, cfg.K, cfg.dtype, cfg.act, cfg.renorm,
                                max_tokens=cfg.T) for _ in range(copies)]
        layers[0].set_router(d_Wr, enorm)
        layers[0].set_resident(first, *arenas[0])
        layers[0].forward(d_x[0], d_out[0])
        imp = layers[0].read_importance(reset=True)
        s2e = binding.topk_importance(imp, cfg.K)
        a_in, a_out = I.build_arena(cfg, s2e)
        arenas = [(dev(a_in), dev(a_out)) for _ in range(copies)]
        del a_in, a_out
        for L, ar in zip(layers, arenas):
            L.set_router(d_Wr, enorm)
            L.set_resident(s2e, *ar)
        layers[0].forward(d_x[0], d_out[0])
        count = layers[0].tap("count")
        uidx = layers[0].tap("uidx")
        for L in layers:
            L.read_importance(reset=True)
            L.read_touched_slots(reset=True)
    touched = int(np.count_nonzero(count))
    hit = float(np.mean(np.isin(uidx, s2e)))

    def step(i, st=stream):
        j = i % copies
        layers[j].forward(d_x[j], d_out[j], stream=st)

    # ---- timed region 1: device-resident inputs
    with torch.cuda.stream(stream):
        for i in range(warmup):
            step(i)
    barrier()
    l0 = sum(L.launch_count for L in layers)
    step(0)
    per_step_launches = sum(L.launch_count for L in layers) - l0
    graph = warm_graph = None
    if not no_graph:
        # One CUDA graph = one rotation over the `copies` replicas (`copies` steps); the timed
        # loop replays it.  forward() neither synchronises nor allocates, so it captures as is.
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream, capture_error_mode="thread_local"):
            for j in range(copies):
                step(j, st=None)
        warm_graph = torch.cuda.CUDAGraph()       # the same number of steps on ONE replica: weights stay in L2 if they fit
        with torch.cuda.graph(warm_graph, stream=stream, capture_error_mode="thread_local"):
            for j in range(copies):
                step(0, st=None)
        for _ in range(3):
            graph.replay()

    def run_steps(g):
        if g is not None:
            for _ in range(steps // copies):
                g.replay()
            for i in range(steps % copies):
                step(i if g is graph else 0)
        else:
            for i in range(steps):
                step(i if g is graph else 0)

    def timed(g, reps):
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
        with torch.cuda.stream(stream):
            evs[0].record(stream)
            for r in range(reps):
                run_steps(g)
                evs[r + 1].record(stream)
        barrier()
        return [evs[r].elapsed_time(evs[r + 1]) for r in range(reps)]

    barrier()
    est = timed(graph, 1)[0]                                      # untimed estimate of one K-step loop
    reps = int(min(400, max(1, np.ceil(min_region_ms / max(est, 1e-3)))))
    if sampler is not None:
        sampler.mark_begin()
    barrier()
    rep_ms = timed(graph, reps)
    ms_total = float(np.median(rep_ms))
    launches = per_step_launches * steps
    warm_ms = float(np.median(timed(warm_graph, max(1, reps // 2)))) if warm_graph is not None else None

    # ---- timed region 2: same steps with events at the stage boundaries (per-kernel times)
    nst = binding.N_STAGES
    n_ev = min(steps, 200)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(nst + 1)] for _ in range(n_ev)]
    with torch.cuda.stream(stream):
        for i in range(n_ev):
            j = i % copies
            layers[j].forward_timed(d_x[j], d_out[j], evs[i], stream=stream)
    barrier()
    stage_ms = np.array([[evs[i][s].elapsed_time(evs[i][s + 1]) for s in range(nst)] for i in range(n_ev)])
    stage_avg = stage_ms.mean(axis=0)

    # ---- timed region 2b: each grouped GEMM alone, launched back to back over the replicas (so its weights come from
    # DRAM every time), two events around the loop: the kernel's duration without the launch gaps the events add
    gemm_alone_ms = None
    try:
        n_al = 25 * copies
        alone = []
        with torch.cuda.stream(stream):
            for j in range(copies):                          # every replica's state is that of its own last forward
                layers[j].forward(d_x[j], d_out[j], stream=stream)
            for which in (1, 2):
                for j in range(copies):
                    layers[j].rerun_gemm(d_out[j], which, stream=stream)
                ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                ea.record(stream)
                for i in range(n_al):
                    layers[i % copies].rerun_gemm(d_out[i % copies], which, stream=stream)
                eb.record(stream)
                alone.append((ea, eb))
        barrier()
        gemm_alone_ms = [a.elapsed_time(b) / n_al for a, b in alone]
    except binding.SwapMoEError:
        gemm_alone_ms = None                                 # paths without a GEMM launch of their own

    out = {"ms_total": ms_total, "rep_ms": rep_ms, "reps": reps, "launches": int(launches), "copies": copies,
           "gemm_alone_ms": gemm_alone_ms,
           "graph": graph is not None, "touched": touched, "count": count, "hit": hit, "warm_ms_total": warm_ms,
           "stage_avg": stage_avg, "stage_ms": stage_ms, "weight_bytes": weight_bytes}

    # ---- timed region 3: end to end through the host-buffer entry point
    if want_e2e:
        xh = torch.from_numpy(I.bf16_bits(x_host).view(np.int16)).view(torch.bfloat16) \
            if cfg.dtype == I.BF16 else torch.from_numpy(x_host)
        xh = xh.pin_memory()
        ohs = [torch.empty((cfg.T, cfg.d), dtype=tdt).pin_memory() for _ in range(copies)]
        # Requests are pipelined over the `copies` layer objects: while one layer computes, the next
        # one's tokens travel host->device and the previous one's result device->host.
        for i in range(3 * copies):
            layers[i % copies].forward_host_async(xh, ohs[i % copies], stream=stream)
        for L in layers:
            L.host_wait()
        barrier()
        e2e_reps = []
        for r in range(max(1, min(reps, 20))):
            t0 = time.perf_counter()
            for i in range(steps):
                layers[i % copies].forward_host_async(xh, ohs[i % copies], stream=stream)
            for L in layers:
                L.host_wait()
            e2e_reps.append(time.perf_counter() - t0)
        barrier()
        # one synchronous request, for the latency of the whole round trip
        t1 = time.perf_counter()
        for i in range(20):
            layers[i % copies].forward_host(xh, ohs[i % copies], stream=stream)
        out["e2e_s"] = float(np.median(e2e_reps))
        out["e2e_sync_ms"] = (time.perf_counter() - t1) / 20 * 1e3
    st = [L.device_status() for L in layers]
    if any(s_[0] != 0 for s_ in st):
        raise SystemExit("device status error: %r" % (st,))
    return out


def layer_entry(cfg, m, steps, peaks, world=1):
    """The figures of one measured configuration, as they go into the JSON line."""
    ms_step = m["ms_total"] / steps
    # average duration of one grouped-GEMM launch: each kernel alone, back to back over the replicas; where the path
    # has no such launch, the stage events of the whole forward (which add a launch gap per stage)
    g_stage = float(m["stage_avg"][3] + m["stage_avg"][4]) / 2.0
    alone = m.get("gemm_alone_ms")
    g_ms = float(sum(alone) / 2.0) if alone else g_stage
    roof, layer = roofline_objects(cfg, m["touched"], g_ms, ms_step, peaks)
    roof["launch_timing"] = ("each grouped GEMM launched alone, back to back over the %d replicas, events around "
                             "%d launches" % (m["copies"], 25 * m["copies"])) if alone else "stage events of the whole forward"
    roof["gemm_alone_us"] = [float(v * 1e3) for v in alone] if alone else None
    roof["stage_event_avg_launch_ms"] = g_stage
    roof["frac_by_stage_events"] = roof["frac"] * g_ms / g_stage
    from paper_2308_15030_b200 import binding
    return {
        "workload": workload_string(cfg), "dtype": "bf16" if cfg.dtype == I.BF16 else "f32",
        "ms_per_step": ms_step, "tokens_per_s": world * cfg.T * steps / (m["ms_total"] * 1e-3),
        "steps": steps, "repeats": m["reps"], "repeat_ms_min_max": [float(min(m["rep_ms"])), float(max(m["rep_ms"]))],
        "warm_ms_per_step": (m["warm_ms_total"] / steps) if m["warm_ms_total"] else None,
        "gpu_launches": m["launches"], "touched_slots": m["touched"], "slot_counts": [int(c) for c in m["count"]],
        "unmasked_hit_rate": m["hit"],
        "l2": "inputs rotate over %d copies of tokens+weights (%.0f MB > 126 MB L2); warm_ms_per_step = the same "
              "loop on one copy" % (m["copies"], m["copies"] * m["weight_bytes"] / 1e6),
        "launch": ("CUDA graph of %d steps, replayed" % m["copies"]) if m["graph"] else "eager",
        "roofline": roof, "layer_roofline": layer,
        "stage_us": {n: float(v * 1e3) for n, v in zip(binding.STAGE_NAMES, m["stage_avg"])},
        "stage_pass_ms_per_step": float(m["stage_ms"].sum(axis=1).mean()),
    }


def run_cuda(args, cfg):
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit("--gpus %d but WORLD_SIZE=%d (launch with torch.distributed.run)" % (args.gpus, world))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()          # started early: nvidia-smi needs a moment before its first sample
    m = measure_layer(cfg, args.steps, args.warmup, rank=rank, world=world, local=local, no_graph=args.no_graph,
                      want_e2e=True, sampler=sampler, barrier=barrier, min_region_ms=args.min_region_ms)
    clocks = sampler.stop() if rank == 0 else None     # sampled over the timed regions (all under load)

    from paper_2308_15030_b200.replicas import max_over_ranks
    ms_total, e2e_ms = max_over_ranks([m["ms_total"], m["e2e_s"] * 1e3], device="cuda")
    m["ms_total"] = ms_total
    if world > 1:
        dist.barrier()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return None

    peaks = load_peaks()
    ent = layer_entry(cfg, m, args.steps, peaks, world)
    res = {
        "metric": METRIC, "value": ent["tokens_per_s"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ent["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": ent["dtype"], "data": "synthetic",
        "config": {"workload": ent["workload"], "l2": ent["l2"], "launch": ent["launch"],
                   "timing": "median of %d back-to-back repeats of the %d-step loop (>= %.0f ms of device time)"
                             % (m["reps"], args.steps, args.min_region_ms),
                   "resident_set": "top-K by Eq.(1) importance of the batch",
                   "touched_slots": ent["touched_slots"], "slot_counts": ent["slot_counts"],
                   "unmasked_hit_rate": ent["unmasked_hit_rate"], "multi_gpu": "replicas only"},
        # kernels of this library launched by the K steps of one timed loop (4 per forward for a bf16 top-1 layer),
        # and over all the repeats of that loop that were timed
        "gpu_launches": ent["gpu_launches"], "gpu_launches_all_repeats": ent["gpu_launches"] * m["reps"],
        "repeats": m["reps"], "repeat_ms_min_max": ent["repeat_ms_min_max"],
        "warm_ms_per_step": ent["warm_ms_per_step"],
        "clocks": clocks,
        "e2e": {"value": world * cfg.T * args.steps / (e2e_ms * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": cfg.T * cfg.d * cfg.nb, "d2h_bytes_per_step": cfg.T * cfg.d * cfg.nb,
                "ms_per_step": e2e_ms / args.steps, "mode": "pipelined over %d layer objects "
                "(swapmoe_forward_host_async)" % m["copies"], "sync_request_ms": m["e2e_sync_ms"]},
        "roofline": ent["roofline"], "layer_roofline": ent["layer_roofline"],
        "stage_us": ent["stage_us"], "stage_pass_ms_per_step": ent["stage_pass_ms_per_step"],
    }
    if world > 1:
        dist.destroy_process_group()
    return res


def run_per_config(args, peaks):
    """Short runs of the other named configurations in the same process (1 GPU): cfg1, cfg3, cfg5 as single
    layers, cfg4 as the decode loop at B = 1, 16, 64 with swapping on and off."""
    import gc
    import torch
    out = {}
    for name, steps in (("cfg1", 200), ("cfg3", 100), ("cfg5", 16)):
        cfg = I.CONFIGS[name]
        sampler = ClockSampler(0)
        sampler.start()
        m = measure_layer(cfg, steps, 5, want_e2e=False, sampler=sampler)
        ent = layer_entry(cfg, m, steps, peaks)
        ent["clocks"] = sampler.stop()
        out[name] = ent
        del m
        gc.collect()
        torch.cuda.empty_cache()
    dargs = argparse.Namespace(**vars(args))
    dargs.steps, dargs.batches, dargs.sweep_frequency, dargs.sweep_budget, dargs.policies = None, [1, 16, 64], None, None, False
    dargs.cfg4_variant = "full"
    d = run_decode(dargs, I.CONFIGS["cfg4"])
    out["cfg4"] = {"workload": d["config"]["workload"], "pcie_probe_GBps": d["pcie_probe_GBps"],
                   "per_batch": d["per_batch"], "clocks": d.get("clocks")}
    return out


# ----------------------------------------------------------------------------- decode loop (cfg4)
def run_decode(args, cfg):
    """12-layer decode loop with asynchronous expert swapping; B tokens per step, 256 steps, every step one CUDA
    graph of the 12 forwards.  Per batch size two arms of the SAME loop: swapping on (importance read every
    `frequency` steps, a global per-step load budget sized from the probed PCIe rate, a slot flips once its copy
    has landed) and the scheduler off.  Each arm reports its own time, the slots its forwards touched (counted
    on the device during that very run) and the roofline fraction that follows."""
    import torch
    from paper_2308_15030_b200 import binding
    from paper_2308_15030_b200.decode import DecodeStack, LayerState, suggest_step_budget
    torch.cuda.set_device(0)
    L, steps, spare = cfg.n_layers, (args.steps or cfg.n_steps), 2
    peaks = load_peaks()
    sampler = ClockSampler(0)
    sampler.start()

    def dev(a):
        return torch.from_numpy(I.bf16_bits(np.ascontiguousarray(a, np.float32)).view(np.int16)).view(torch.bfloat16).cuda()

    # PCIe probe: 1 GiB pinned -> device, best of 10
    probe_h = torch.empty(1 << 30, dtype=torch.uint8).pin_memory()
    probe_d = torch.empty(1 << 30, dtype=torch.uint8, device="cuda")
    best = 1e9
    for _ in range(10):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); probe_d.copy_(probe_h, non_blocking=True); b.record(); b.synchronize()
        best = min(best, a.elapsed_time(b))
    pcie_gbs = (1 << 30) / (best * 1e-3) / 1e9
    del probe_h, probe_d

    # One bank of E experts (values shared by the layers: only timing is measured here), one
    # pinned copy per layer so every layer's loads come from its own host memory.
    w_in = np.empty((cfg.E, cfg.nin, cfg.f, cfg.d), np.float32)
    w_out = np.empty((cfg.E, cfg.d, cfg.f), np.float32)
    for e in range(cfg.E):
        w_in[e], w_out[e] = I.make_expert(cfg, e)
    bank_in = torch.from_numpy(I.bf16_bits(w_in).view(np.int16)).view(torch.bfloat16)
    bank_out = torch.from_numpy(I.bf16_bits(w_out).view(np.int16)).view(torch.bfloat16)
    del w_in, w_out
    host_in = [bank_in.clone().pin_memory() for _ in range(L)]
    host_out = [bank_out.clone().pin_memory() for _ in range(L)]
    Wr = [I.make_router(cfg.scaled(seed=1000 + l)) for l in range(L)]
    enorm = [I.make_enorm(cfg.scaled(seed=1000 + l)) for l in range(L)]
    d_Wr = [dev(w) for w in Wr]
    expert_bytes = cfg.nmat * cfg.d * cfg.f * cfg.nb
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    results = {}
    first_timed = True
    for B in args.batches:
        x = I.make_decode_tokens(cfg, Wr, B, steps)
        d_x = dev(x.reshape(-1, cfg.d)).reshape(steps, L, B, cfg.d)
        outs = torch.empty((L, B, cfg.d), dtype=torch.bfloat16, device="cuda")
        xbuf = torch.empty((L, B, cfg.d), dtype=torch.bfloat16, device="cuda")

        def make_stack(Ks=None, **kw):
            states = []
            for l in range(L):
                K = cfg.K if Ks is None else Ks[l]
                P = K + spare
                a_in = torch.empty((P, cfg.nin, cfg.f, cfg.d), dtype=torch.bfloat16, device="cuda")
                a_out = torch.empty((P, cfg.d, cfg.f), dtype=torch.bfloat16, device="cuda")
                a_in[:K].copy_(host_in[l][:K]); a_out[:K].copy_(host_out[l][:K])
                layer = binding.Layer(cfg.E, cfg.d, cfg.f, cfg.k, K, cfg.dtype, cfg.act, cfg.renorm,
                                      max_tokens=B, spare_slots=spare)
                layer.set_router(d_Wr[l], enorm[l])
                states.append(LayerState(layer, np.arange(K, dtype=np.int32), np.arange(K, dtype=np.int32),
                                         list(range(K, P)), a_in, a_out, host_in[l], host_out[l], enorm=enorm[l]))
            torch.cuda.synchronize()
            kw.setdefault("lag", 2)
            return DecodeStack(states, graph_buffers=(xbuf, outs), **kw)

        def run_arm(stack, graph=True):
            """Warm-up of 8 steps (tables evolve; they are part of the loop), then the timed loop."""
            nonlocal first_timed
            stepper = (lambda s_: stack.step_graph(d_x[s_])) if graph else \
                (lambda s_: stack.step([d_x[s_, l] for l in range(L)], [outs[l] for l in range(L)], record=False))
            for s_ in range(min(8, steps)):
                stepper(s_)
            torch.cuda.synchronize()
            for st in stack.layers:
                st.layer.read_touched_slots(reset=True)
                st.layer.read_decode_prefetch(reset=True)
            base = dict(host=stack.host_seconds, waits=stack.throttle_waits, loads=stack.loads, bytes=stack.bytes_loaded, stalls=stack.stalls, deferred=stack.deferred,
                        commits=stack.commits, hits=stack.hits, asked=stack.asked, misses=stack.misses,
                        blocking=stack.blocking_loads, requests=stack.requests, n_ev=len(stack.load_events),
                        launches=sum(st.layer.launch_count for st in stack.layers), replays=stack.graph_replays)
            if first_timed:
                sampler.mark_begin()
                first_timed = False
            gc.collect(); gc.disable()           # no collector pause inside the timed loop (the scheduler is Python)
            e0.record()
            for s_ in range(steps):
                stepper(s_)
            e1.record(); torch.cuda.synchronize()
            gc.enable()
            ms = e0.elapsed_time(e1)
            touched = sum(st.layer.read_touched_slots(reset=True) for st in stack.layers)
            pf = [st.layer.read_decode_prefetch(reset=True) for st in stack.layers]
            status = [st.layer.device_status() for st in stack.layers]
            assert all(s_ == (0, 0) for s_ in status), status
            bytes_alg = touched * expert_bytes + steps * L * (2 * B * cfg.d * cfg.nb + cfg.E * cfg.d * cfg.nb)
            t_roof = bytes_alg / (peaks["hbm_gbs"] * 1e9)
            load_s = sum(a.elapsed_time(b) for a, b in stack.load_events[base["n_ev"]:]) * 1e-3
            nbytes = stack.bytes_loaded - base["bytes"]
            r = {"tokens_per_s": steps * B / (ms * 1e-3), "ms_per_step": ms / steps, "us_per_layer": ms / steps / L * 1e3,
                 # eager launches (score snapshots, table updates) + the kernels of every replay of the captured step
                 "gpu_launches": sum(st.layer.launch_count for st in stack.layers) - base["launches"]
                 + (stack.graph_replays - base["replays"]) * stack.graph_launches,
                 "touched_slots_per_layer_step": touched / (steps * L),
                 "roofline_us_per_layer": t_roof / (steps * L) * 1e6, "roofline_frac": t_roof * 1e3 / ms,
                 "loads": stack.loads - base["loads"], "loaded_GB": nbytes / 1e9,
                 "commits": stack.commits - base["commits"], "stalls": stack.stalls - base["stalls"],
                 "deferred_commits": stack.deferred - base["deferred"],
                 "pcie_seconds_needed": nbytes / (pcie_gbs * 1e9), "loop_seconds": ms * 1e-3,
                 # host time per step spent preparing and enqueuing (waiting for the device excluded), and the share
                 # of steps before which the device was still busy (else the loop is bound by the host)
                 "host_ms_per_step": (stack.host_seconds - base["host"]) / steps * 1e3,
                 "steps_host_waited_for_device": (stack.throttle_waits - base["waits"]) / steps}
            if sum(t_ for _, t_ in pf) > 0:      # one-launch decode steps: L2 prefetch of the recently served experts
                r["decode_prefetch_hit_rate"] = sum(h_ for h_, _ in pf) / sum(t_ for _, t_ in pf)
            if load_s > 0:
                r["loader_GBps"] = nbytes / load_s / 1e9
                r["loader_frac_of_pcie_probe"] = nbytes / load_s / 1e9 / pcie_gbs
            if stack.asked > base["asked"]:
                r["resident_hit_rate"] = (stack.hits - base["hits"]) / (stack.asked - base["asked"])
            if stack.requests > base["requests"]:
                r["miss_rate"] = (stack.misses - base["misses"]) / (stack.requests - base["requests"])
                r["blocking_loads"] = stack.blocking_loads - base["blocking"]
            return r

        # arm 1: scheduler off (no importance reads, no swaps): what the kernels alone allow
        no_swap = run_arm(make_stack(frequency=1 << 30, max_in_flight=3))
        # the host may run ahead of the device by about 1.5 ms of queued steps (at least 3, at most 8 steps): enough to
        # ride out a step in which the scheduler decides, short enough for its decisions to be current
        mif = args.max_in_flight or max(3, min(8, int(1.5e-3 / (no_swap["ms_per_step"] * 1e-3))))
        # arm 2: swapping on.  The step's load budget follows the link: what PCIe carries while a step computes.
        budget = suggest_step_budget(no_swap["ms_per_step"] * 1e-3, pcie_gbs, expert_bytes)
        if args.cfg4_variant == "no_loads":          # diagnostic: decisions only
            budget = 0.0
        swap = run_arm(make_stack(frequency=args.frequency, loads_per_step=1, step_budget=budget, commit="ready",
                                  lag=(10 ** 9 if args.cfg4_variant == "no_commits" else 2),
                                  time_loads=(B == max(args.batches)), track_hits=True, async_decide=True,
                                  max_in_flight=mif))
        swap["step_budget"] = budget
        swap["max_in_flight"] = mif
        swap["slowdown_vs_no_swap"] = swap["us_per_layer"] / no_swap["us_per_layer"]
        entry = {"swap": swap, "no_swap": no_swap}
        big = B == max(args.batches)
        # Section 3.4.1: sweep the update frequency (rare -> frequent) and the loads per step
        if args.sweep_frequency and big:
            entry["frequency_sweep"] = {
                str(fr): run_arm(make_stack(frequency=fr, loads_per_step=1, step_budget=budget, commit="ready",
                                            track_hits=True, async_decide=True, max_in_flight=mif)) for fr in args.sweep_frequency}
        if args.sweep_budget and big:
            entry["budget_sweep"] = {
                ("%g" % bu): run_arm(make_stack(frequency=args.frequency, loads_per_step=max(1, int(-(-bu // L))), step_budget=bu,
                                            commit="wait" if args.sweep_commit == "wait" else "ready", track_hits=True,
                                            async_decide=True, max_in_flight=mif))
                for bu in args.sweep_budget}
        # Section 4.1 baselines as policies over the same kernels, and per-layer budgets (Section 3.3)
        if args.policies and big:
            pol = {}
            for K in (4, 8, 16):
                Ks = [K] * L
                pol["K=%d" % K] = {
                    "swap": run_arm(make_stack(Ks, frequency=args.frequency, loads_per_step=1, step_budget=budget,
                                               commit="ready", track_hits=True, async_decide=True, max_in_flight=mif)),
                    "static_pruning": run_arm(make_stack(Ks, policy="static_pruning")),
                    "on_demand": run_arm(make_stack(Ks, policy="on_demand", lag=0), graph=False)}
            entry["policies_vs_K"] = pol
            Ks = [8, 12, 16, 24] * (L // 4) + [16] * (L % 4)
            entry["per_layer_K"] = dict(run_arm(make_stack(Ks, frequency=args.frequency, loads_per_step=1,
                                                           step_budget=budget, commit="ready", track_hits=True,
                                                           async_decide=True, max_in_flight=mif)), Ks=Ks)
        results[str(B)] = entry
    clocks = sampler.stop()
    Bmax = str(max(args.batches))
    top = results[Bmax]["swap"]
    return {
        "metric": METRIC, "value": top["tokens_per_s"], "unit": UNIT, "n_gpus": 1, "steps": steps,
        "warmup": 8, "ms_per_step": top["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "cfg4 decode loop: %d layers d_model=%d d_ff=%d E=%d top1 K=%d, %d steps, "
                               "B in %s tokens per step; swapping on: importance read every %d steps, global load "
                               "budget per step from the PCIe probe, a slot flips once its copy has landed, %d spare "
                               "slots; value = B=%s" % (L, cfg.d, cfg.f, cfg.E, cfg.K, steps, args.batches,
                                                        args.frequency, spare, Bmax),
                   "expert_bank": "one bank of %d experts, copied into %d per-layer pinned buffers" % (cfg.E, L),
                   "launch": "one CUDA graph per step (12 forwards); table flips and copies outside it",
                   "l2": "per-step weight traffic (touched slots x 16.8 MB x 12 layers) exceeds the 126 MB L2"},
        "gpu_launches": top["gpu_launches"],
        # the same arm as `value`: the whole step with swapping on, against the HBM time of the slots it touched
        "roofline": {"bound": "hbm", "unit": "GB/s", "peak": peaks["hbm_gbs"], "peak_source": peaks["source"],
                     "achieved": peaks["hbm_gbs"] * top["roofline_frac"], "frac": top["roofline_frac"], "traffic": None,
                     "kernel": "whole layer forward (router .. combine), B = %s, swapping on" % Bmax,
                     "frac_scheduler_off": results[Bmax]["no_swap"]["roofline_frac"]},
        "clocks": clocks, "pcie_probe_GBps": pcie_gbs, "per_batch": results,
    }


# ----------------------------------------------------------------------------- the oracle arm
def oracle_sample(cfg, steps=1, warmup=0, budget_s=None):
    """Times the CPU oracle, as it stands, on the workload's batch (host cores)."""
    import oracle
    Wr = I.make_router(cfg)
    enorm = I.make_enorm(cfg)
    x = I.make_tokens(cfg, Wr)
    lg = oracle.logits(x, Wr)
    uidx, ugate = oracle.gate(lg, cfg.k, cfg.renorm)
    s2e = oracle.topk_importance(oracle.importance(x, uidx, ugate, enorm), cfg.K)
    a_in, a_out = I.build_arena(cfg, s2e)
    # bound the work to roughly 10-30 s: the FFN of a token subset, routing over all tokens
    flops_tok = 2.0 * cfg.k * cfg.d * cfg.f * cfg.nmat
    n_sub = int(min(cfg.T, max(16, 40e9 / flops_tok)))
    sub = None if n_sub >= cfg.T else np.sort(
        np.random.default_rng(0).choice(cfg.T, n_sub, replace=False)).astype(np.int32)
    times = []
    t_begin = time.perf_counter()
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        oracle.forward(x, Wr, enorm, s2e, a_in, a_out, k=cfg.k, act=cfg.act, renorm=cfg.renorm,
                       token_subset=sub)
        dt = time.perf_counter() - t0
        if i >= warmup:
            times.append(dt)
        # the asked-for steps are honoured while the whole run stays within the budget
        if budget_s is not None and times and (time.perf_counter() - t_begin) + dt > budget_s:
            break
    n_tok = cfg.T if sub is None else n_sub
    sample = ("full %d-token batch" % cfg.T) if sub is None else \
        ("routing on all %d tokens, expert FFN on a seeded %d-token subset; tokens/s counts the subset"
         % (cfg.T, n_sub))
    return n_tok, times, oracle.num_threads(), sample


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return None
    # --steps / --warmup are honoured as long as the run is estimated to stay under a minute
    n_tok, times, cores, sample = oracle_sample(cfg, steps=args.steps, warmup=args.warmup, budget_s=60.0)
    total = float(np.sum(times))
    value = n_tok * len(times) / total
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": len(times), "steps_asked": args.steps, "warmup": args.warmup, "ms_per_step": total / len(times) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": workload_string(cfg)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
    ap.add_argument("--batches", type=int, nargs="+", default=[1, 4, 16, 64], help="cfg4: tokens per decode step")
    ap.add_argument("--frequency", type=int, default=8, help="cfg4: steps between two updates of the resident sets")
    ap.add_argument("--sweep-frequency", type=int, nargs="*", default=None,
                    help="cfg4: also run the loop (largest batch) at these update frequencies (steps between updates)")
    ap.add_argument("--sweep-budget", type=float, nargs="*", default=None,
                    help="cfg4: also run the loop (largest batch) with these numbers of expert loads per step")
    ap.add_argument("--sweep-commit", default="ready", choices=["ready", "wait"],
                    help="cfg4 budget sweep: flip when the copy has landed, or wait for it at the commit step")
    ap.add_argument("--cfg4-variant", default="full", choices=["full", "no_loads", "no_commits"],
                    help="cfg4 diagnostic: swapping arm without expert copies / with copies that are never committed")
    ap.add_argument("--max-in-flight", type=int, default=0,
                    help="cfg4: steps the host may run ahead of the device in the swapping arms (0: from the step time)")
    ap.add_argument("--policies", action="store_true",
                    help="cfg4: also run static pruning / on-demand loading / swapping at K = 4, 8, 16 and per-layer K")
    ap.add_argument("--min-region-ms", type=float, default=MIN_REGION_MS,
                    help="repeat the timed K-step loop until it covers this much device time (0: once; for profiler runs)")
    ap.add_argument("--no-per-config", action="store_true",
                    help="default workload: skip the short runs of cfg1, cfg3, cfg4, cfg5 that fill `per_config`")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch every step eagerly instead of replaying a CUDA graph")
    args = ap.parse_args()
    cfg = I.CONFIGS[args.workload]
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        res = run_reference(args, cfg)
        if res is not None:
            print(json.dumps(res), flush=True)
        return
    if args.workload == "cfg4":
        print(json.dumps(run_decode(args, cfg)), flush=True)
        return
    per_config = args.workload == "cfg2" and args.gpus == 1 and not args.no_per_config
    args.steps = 2000 if args.steps is None else args.steps
    args.warmup = 50 if args.warmup is None else max(3, args.warmup)
    res = run_cuda(args, cfg)
    if res is None:
        return
    if per_config:
        res["per_config"] = run_per_config(args, load_peaks())
    if args.gpus == 1 and not args.no_cpu_baseline:
        n_tok, times, cores, sample = oracle_sample(cfg, steps=3, warmup=0)
        res["cpu_baseline"] = {"value": n_tok / float(np.min(times)), "unit": UNIT, "cores": cores,
                               "kind": "oracle", "sample": sample}
    print(json.dumps(res), flush=True)


if __name__ == "__main__":
    main()
