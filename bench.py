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

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the grouped-GEMM kernel, mean of the
# GEMM-1 and GEMM-2 launches of one step, from the ncu capture summarised in
# profiles/cfg2_router_permute_tc_gemm.md (80.07 + 5.99 MB and 93.63 + 3.65 MB).
NCU_TRAFFIC_PER_LAUNCH = {"cfg2": (80.07e6 + 5.99e6 + 93.63e6 + 3.65e6) / 2}

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


def run_cuda(args, cfg):
    import torch
    import torch.distributed as dist
    from paper_2308_15030_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit("--gpus %d but WORLD_SIZE=%d (launch with torch.distributed.run)" % (args.gpus, world))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    tdt = torch.bfloat16 if cfg.dtype == I.BF16 else torch.float32

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
    touched = int(np.count_nonzero(count))
    hit = float(np.mean(np.isin(uidx, s2e)))

    def step(i, st=stream):
        j = i % copies
        layers[j].forward(d_x[j], d_out[j], stream=st)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()          # started early: nvidia-smi needs a moment before its first sample
    # ---- timed region 1: device-resident inputs
    with torch.cuda.stream(stream):
        for i in range(args.warmup):
            step(i)
    barrier()
    l0 = sum(L.launch_count for L in layers)
    step(0)
    per_step_launches = sum(L.launch_count for L in layers) - l0
    graph = None
    if not args.no_graph:
        # One CUDA graph = one rotation over the `copies` replicas (`copies` steps); the timed
        # loop replays it.  forward() neither synchronises nor allocates, so it captures as is.
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream, capture_error_mode="thread_local"):
            for j in range(copies):
                step(j, st=None)
        for _ in range(3):
            graph.replay()
    barrier()
    sampler.mark_begin()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    with torch.cuda.stream(stream):
        e0.record(stream)
        if graph is not None:
            for _ in range(args.steps // copies):
                graph.replay()
            for i in range(args.steps % copies):
                step(i)
        else:
            for i in range(args.steps):
                step(i)
        e1.record(stream)
    barrier()
    ms_total = e0.elapsed_time(e1)
    launches = per_step_launches * args.steps

    # ---- timed region 2: same steps with events at the stage boundaries (per-kernel times)
    nst = binding.N_STAGES
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(nst + 1)] for _ in range(args.steps)]
    with torch.cuda.stream(stream):
        for i in range(args.steps):
            j = i % copies
            layers[j].forward_timed(d_x[j], d_out[j], evs[i], stream=stream)
    barrier()
    stage_ms = np.array([[evs[i][s].elapsed_time(evs[i][s + 1]) for s in range(nst)]
                         for i in range(args.steps)])
    stage_avg = stage_ms.mean(axis=0)

    # ---- timed region 3: end to end through the host-buffer entry point
    xh = torch.from_numpy(I.bf16_bits(x_host).view(np.int16)).view(torch.bfloat16) \
        if cfg.dtype == I.BF16 else torch.from_numpy(x_host)
    xh = xh.pin_memory()
    ohs = [torch.empty((cfg.T, cfg.d), dtype=tdt).pin_memory() for _ in range(copies)]
    # Requests are pipelined over the `copies` layer objects: while one layer computes, the next
    # one's tokens travel host->device and the previous one's result device->host.
    for i in range(min(3, args.warmup) * copies):
        layers[i % copies].forward_host_async(xh, ohs[i % copies], stream=stream)
    for L in layers:
        L.host_wait()
    barrier()
    t0 = time.perf_counter()
    for i in range(args.steps):
        layers[i % copies].forward_host_async(xh, ohs[i % copies], stream=stream)
    for L in layers:
        L.host_wait()
    barrier()
    e2e_s = time.perf_counter() - t0
    # one synchronous request, for the latency of the whole round trip
    t1 = time.perf_counter()
    for i in range(20):
        layers[i % copies].forward_host(xh, ohs[i % copies], stream=stream)
    e2e_sync_ms = (time.perf_counter() - t1) / 20 * 1e3

    clocks = sampler.stop() if rank == 0 else None     # sampled over all three timed regions (all under load)
    st = [L.device_status() for L in layers]
    if any(s[0] != 0 for s in st):
        raise SystemExit("device status error: %r" % (st,))

    from paper_2308_15030_b200.replicas import max_over_ranks
    ms_total, e2e_ms = max_over_ranks([ms_total, e2e_s * 1e3], device="cuda")
    if world > 1:
        dist.barrier()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return None

    peaks = load_peaks()
    ms_step = ms_total / args.steps
    value = world * cfg.T * args.steps / (ms_total * 1e-3)
    g_bytes, g_flops = gemm_algorithmic(cfg, touched)
    g_ms = float(stage_avg[3] + stage_avg[4]) / 2.0          # average duration of one GEMM launch
    # Tensor peak: kernels timed inside a long, power-capped step (>= 1 ms per step) are held against
    # the sustained cuBLAS figure, short ones against the burst figure.
    tc_kind = "sustained" if ms_step >= 1.0 else "burst"
    tc_peak = peaks["bf16_tflops_sustained"] if tc_kind == "sustained" else peaks["bf16_tflops"]
    t_hbm = g_bytes / (peaks["hbm_gbs"] * 1e9)
    t_tc = g_flops / (tc_peak * 1e12) if cfg.dtype == I.BF16 else 0.0
    ffma = os.environ.get("SWAPMOE_FP32_FFMA") == "1"
    # fp32 layers: the grouped GEMM runs on the tensor cores as three TF32 products per fp32 product;
    # its peak is the measured bf16 figure x the nominal TF32 : bf16 ratio (1.1 : 2.25 PFLOP/s) / 3.
    # (With SWAPMOE_FP32_FFMA=1 it is an FFMA kernel: 148 SMs x 128 lanes x 2 x 1.965 GHz = 74.4 TFLOP/s.)
    tf32x3_peak = peaks["bf16_tflops"] * (1.1 / 2.25) / 3.0
    if cfg.dtype != I.BF16 and ffma:
        bound, peak, ach, unit = "alu", 74.4, g_flops / 2 / (g_ms * 1e-3) / 1e12, "TFLOP/s"
    elif cfg.dtype != I.BF16 and t_hbm >= g_flops / (tf32x3_peak * 1e12):
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
                 layer_flops / (tc_peak * 1e12) if cfg.dtype == I.BF16
                 else layer_flops / ((74.4 if ffma else tf32x3_peak) * 1e12))
    res = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if cfg.dtype == I.BF16 else "f32", "data": "synthetic",
        "config": {"workload": workload_string(cfg),
                   "l2": "inputs rotate over %d copies of tokens+weights (%.0f MB > 126 MB L2)"
                         % (copies, copies * weight_bytes / 1e6),
                   "launch": ("CUDA graph of %d steps, replayed" % copies) if graph is not None else "eager",
                   "resident_set": "top-K by Eq.(1) importance of the batch",
                   "touched_slots": touched, "slot_counts": [int(c) for c in count],
                   "unmasked_hit_rate": hit, "multi_gpu": "replicas only"},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "e2e": {"value": world * cfg.T * args.steps / (e2e_ms * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": cfg.T * cfg.d * cfg.nb, "d2h_bytes_per_step": cfg.T * cfg.d * cfg.nb,
                "ms_per_step": e2e_ms / args.steps, "mode": "pipelined over %d layer objects "
                "(swapmoe_forward_host_async)" % copies, "sync_request_ms": e2e_sync_ms},
        "roofline": {"bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak,
                     "traffic": NCU_TRAFFIC_PER_LAUNCH.get(cfg.name), "peak_source": peaks["source"],
                     "kernel": "tc_gemm_kernel (grouped FFN GEMM, 2 launches per step: GEMM-1+act, GEMM-2)"
                               if cfg.dtype == I.BF16 else ("gemm_simt_kernel (FFMA, 2 launches per step)" if ffma else
                                                            ("gemm_tf32x3_kernel (split-TF32 warp-level mma, 2 launches per step)"
                                                             if os.environ.get("SWAPMOE_FP32_TC") == "0" else
                                                             "tc_gemm_f32_kernel (split-TF32 on tcgen05, 2 launches per step)")),
                     "algorithmic_bytes_per_launch": g_bytes / 2, "flops_per_launch": g_flops / 2,
                     "avg_launch_ms": g_ms,
                     "tensor_tflops": g_flops / 2 / (g_ms * 1e-3) / 1e12,
                     "tensor_peak_kind": (tc_kind if cfg.dtype == I.BF16 else "bf16 burst x 1.1/2.25 / 3 (TF32 x3)")
                                         if bound == "tensor" else None,
                     "frac_of_fp32_ffma_peak": (g_flops / 2 / (g_ms * 1e-3) / 1e12 / 74.4) if cfg.dtype != I.BF16 else None,
                     "frac_of_burst_tensor_peak": (ach / peaks["bf16_tflops"]) if bound == "tensor" else None},
        "layer_roofline": {"t_roof_us": t_roof * 1e6, "frac": t_roof * 1e3 / ms_step,
                           "algorithmic_bytes": layer_bytes, "flops": layer_flops},
        "stage_us": {n: float(v * 1e3) for n, v in zip(binding.STAGE_NAMES, stage_avg)},
        "stage_pass_ms_per_step": float(stage_ms.sum(axis=1).mean()),
    }
    if world > 1:
        dist.destroy_process_group()
    return res


# ----------------------------------------------------------------------------- decode loop (cfg4)
def run_decode(args, cfg):
    """12-layer decode loop with asynchronous expert swapping; B tokens per step, 256 steps.
    Reports tokens/s through the whole stack for each batch size, the achieved host->device
    rate of the expert copies against a PCIe peak probed in the same run, and the stalls."""
    import torch
    from paper_2308_15030_b200 import binding
    from paper_2308_15030_b200.decode import DecodeStack, LayerState
    torch.cuda.set_device(0)
    L, steps, spare = cfg.n_layers, (args.steps or cfg.n_steps), 2
    peaks = load_peaks()

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

    results = {}
    for B in args.batches:
        x = I.make_decode_tokens(cfg, Wr, B, steps)
        d_x = dev(x.reshape(-1, cfg.d)).reshape(steps, L, B, cfg.d)
        outs = torch.empty((L, B, cfg.d), dtype=torch.bfloat16, device="cuda")

        xbuf = torch.empty((L, B, cfg.d), dtype=torch.bfloat16, device="cuda")

        def make_stack(time_loads, frequency=8, graph=False):
            states = []
            for l in range(L):
                P = cfg.K + spare
                a_in = torch.empty((P, cfg.nin, cfg.f, cfg.d), dtype=torch.bfloat16, device="cuda")
                a_out = torch.empty((P, cfg.d, cfg.f), dtype=torch.bfloat16, device="cuda")
                a_in[: cfg.K].copy_(host_in[l][: cfg.K]); a_out[: cfg.K].copy_(host_out[l][: cfg.K])
                layer = binding.Layer(cfg.E, cfg.d, cfg.f, cfg.k, cfg.K, cfg.dtype, cfg.act, cfg.renorm,
                                      max_tokens=B, spare_slots=spare)
                layer.set_router(d_Wr[l], enorm[l])
                states.append(LayerState(layer, np.arange(cfg.K, dtype=np.int32), np.arange(cfg.K, dtype=np.int32),
                                         list(range(cfg.K, P)), a_in, a_out, host_in[l], host_out[l]))
            torch.cuda.synchronize()
            return DecodeStack(states, frequency=frequency, loads_per_step=1, lag=2, time_loads=time_loads,
                               graph_buffers=(xbuf, outs) if graph else None)

        # pass 1: timed, nothing read back except the importance every 8 steps
        stack = make_stack(True)
        for s in range(min(8, steps)):            # warm-up steps (tables evolve; they are part of the loop)
            stack.step([d_x[s, l] for l in range(L)], [outs[l] for l in range(L)], record=False)
        torch.cuda.synchronize()
        stack2_start = stack.step_no
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches0 = sum(st.layer.launch_count for st in stack.layers)
        e0.record()
        for s in range(steps):
            stack.step([d_x[s, l] for l in range(L)], [outs[l] for l in range(L)], record=False)
        e1.record(); torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        launches = sum(st.layer.launch_count for st in stack.layers) - launches0
        load_s = stack.loader_seconds()
        loads, bytes_loaded, stalls = stack.loads, stack.bytes_loaded, stack.stalls
        status = [st.layer.device_status() for st in stack.layers]
        assert all(s == (0, 0) for s in status), status
        del stack
        # pass 1b: the same loop with the scheduler switched off (no importance reads, no swaps):
        # what the kernels alone allow, to separate compute from PCIe traffic
        stack = make_stack(False, frequency=1 << 30)
        for s in range(min(8, steps)):
            stack.step([d_x[s, l] for l in range(L)], [outs[l] for l in range(L)], record=False)
        torch.cuda.synchronize()
        e0.record()
        for s in range(steps):
            stack.step([d_x[s, l] for l in range(L)], [outs[l] for l in range(L)], record=False)
        e1.record(); torch.cuda.synchronize()
        ms_noswap = e0.elapsed_time(e1)
        del stack
        # pass 1c: scheduler off, the step's 12 forwards replayed as one CUDA graph
        stack = make_stack(False, frequency=1 << 30, graph=True)
        for s in range(min(8, steps)):
            stack.step_graph(d_x[s])
        torch.cuda.synchronize()
        e0.record()
        for s in range(steps):
            stack.step_graph(d_x[s])
        e1.record(); torch.cuda.synchronize()
        ms_graph = e0.elapsed_time(e1)
        del stack
        # pass 1d: scheduler ON with the graph
        stack = make_stack(False, frequency=8, graph=True)
        for s in range(min(8, steps)):
            stack.step_graph(d_x[s])
        torch.cuda.synchronize()
        e0.record()
        for s in range(steps):
            stack.step_graph(d_x[s])
        e1.record(); torch.cuda.synchronize()
        ms_graph_swap = e0.elapsed_time(e1)
        del stack
        # pass 1e (optional): Section 3.4.1's search - run the loop at several update frequencies,
        # from rare to frequent updates, and report where swapping starts to cost latency
        sweep = {}
        if args.sweep_frequency and B == max(args.batches):
            for freq in args.sweep_frequency:
                stack = make_stack(False, frequency=freq, graph=True)
                for s in range(min(8, steps)):
                    stack.step_graph(d_x[s])
                torch.cuda.synchronize()
                l0, st0 = stack.loads, stack.stalls
                e0.record()
                for s in range(steps):
                    stack.step_graph(d_x[s])
                e1.record(); torch.cuda.synchronize()
                sweep[str(freq)] = {"us_per_layer": e0.elapsed_time(e1) / steps / L * 1e3,
                                    "loads": stack.loads - l0, "stalls": stack.stalls - st0}
                del stack
        # pass 2: same inputs, slot counts tapped after every forward -> touched slots for the roofline
        stack = make_stack(False)
        touched = 0
        for s in range(min(8, steps)):
            stack.step([d_x[s, l] for l in range(L)], [outs[l] for l in range(L)], record=False)
        for s in range(steps):
            n = stack.step_no
            for li, st in enumerate(stack.layers):
                stack._commit_due(st, n)
                st.layer.forward(d_x[s, li], outs[li])
                touched += int(np.count_nonzero(st.layer.tap("count")))
            if (n + 1) % stack.frequency == 0:
                for li, st in enumerate(stack.layers):
                    stack._decide(li, st, n)
            for st in stack.layers:
                stack._issue_loads(st, n)
            stack.step_no += 1
        torch.cuda.synchronize()
        del stack
        bytes_alg = touched * expert_bytes + steps * L * (2 * B * cfg.d * cfg.nb + cfg.E * cfg.d * cfg.nb)
        t_roof = bytes_alg / (peaks["hbm_gbs"] * 1e9)
        results[str(B)] = {
            "tokens_per_s": steps * B / (ms * 1e-3), "ms_per_step": ms / steps,
            "us_per_layer": ms / steps / L * 1e3, "gpu_launches": int(launches),
            "touched_slots_per_layer_step": touched / (steps * L),
            "roofline_us_per_layer": t_roof / (steps * L) * 1e6, "roofline_frac": t_roof * 1e3 / ms,
            "loads": loads, "loaded_GB": bytes_loaded / 1e9,
            "loader_GBps": (bytes_loaded / load_s / 1e9) if load_s > 0 else None,
            "loader_frac_of_pcie_probe": (bytes_loaded / load_s / 1e9 / pcie_gbs) if load_s > 0 else None,
            "stalls": stalls,
            "pcie_seconds_needed": bytes_loaded / (pcie_gbs * 1e9), "loop_seconds": ms * 1e-3,
            "frequency_sweep": sweep,
            "no_swap": {"tokens_per_s": steps * B / (ms_noswap * 1e-3), "us_per_layer": ms_noswap / steps / L * 1e3},
            "no_swap_graph": {"tokens_per_s": steps * B / (ms_graph * 1e-3), "us_per_layer": ms_graph / steps / L * 1e3,
                              "roofline_frac": t_roof * 1e3 / ms_graph},
            "swap_graph": {"tokens_per_s": steps * B / (ms_graph_swap * 1e-3),
                           "us_per_layer": ms_graph_swap / steps / L * 1e3},
        }
    Bmax = str(max(args.batches))
    return {
        "metric": METRIC, "value": results[Bmax]["tokens_per_s"], "unit": UNIT, "n_gpus": 1, "steps": steps,
        "warmup": 8, "ms_per_step": results[Bmax]["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "cfg4 decode loop: %d layers d_model=%d d_ff=%d E=%d top1 K=%d, %d steps, "
                               "B in %s tokens per step; frequency 8, <=1 load/layer/step, commit lag 2, 2 spare "
                               "slots; value = B=%s" % (L, cfg.d, cfg.f, cfg.E, cfg.K, steps, args.batches, Bmax),
                   "expert_bank": "one bank of %d experts, copied into %d per-layer pinned buffers" % (cfg.E, L),
                   "launch": "eager (host policy in the loop)"},
        "gpu_launches": results[Bmax]["gpu_launches"],
        # the layer kernels with the scheduler off (graph replay), against the HBM time of the touched slots' weights
        "roofline": {"bound": "hbm", "unit": "GB/s", "peak": peaks["hbm_gbs"], "peak_source": peaks["source"],
                     "achieved": peaks["hbm_gbs"] * results[Bmax]["no_swap_graph"]["roofline_frac"],
                     "frac": results[Bmax]["no_swap_graph"]["roofline_frac"], "traffic": None,
                     "kernel": "whole layer forward (router .. combine), B = %s, scheduler off" % Bmax},
        "pcie_probe_GBps": pcie_gbs, "per_batch": results,
    }


# ----------------------------------------------------------------------------- the oracle arm
def oracle_sample(cfg, steps=1, warmup=0):
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
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        oracle.forward(x, Wr, enorm, s2e, a_in, a_out, k=cfg.k, act=cfg.act, renorm=cfg.renorm,
                       token_subset=sub)
        if i >= warmup:
            times.append(time.perf_counter() - t0)
    n_tok = cfg.T if sub is None else n_sub
    sample = ("full %d-token batch" % cfg.T) if sub is None else \
        ("routing on all %d tokens, expert FFN on a seeded %d-token subset; tokens/s counts the subset"
         % (cfg.T, n_sub))
    return n_tok, times, oracle.num_threads(), sample


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return None
    n_tok, times, cores, sample = oracle_sample(cfg, steps=args.steps, warmup=min(args.warmup, 1))
    total = float(np.sum(times))
    value = n_tok * len(times) / total
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": min(args.warmup, 1), "ms_per_step": total / len(times) * 1e3,
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
    ap.add_argument("--sweep-frequency", type=int, nargs="*", default=None,
                    help="cfg4: also run the loop (largest batch) at these update frequencies (steps between updates)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch every step eagerly instead of replaying a CUDA graph")
    args = ap.parse_args()
    cfg = I.CONFIGS[args.workload]
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else min(args.steps, 5)
        args.warmup = 1 if args.warmup is None else args.warmup
        res = run_reference(args, cfg)
        if res is not None:
            print(json.dumps(res), flush=True)
        return
    if args.workload == "cfg4":
        print(json.dumps(run_decode(args, cfg)), flush=True)
        return
    args.steps = 2000 if args.steps is None else args.steps
    args.warmup = 50 if args.warmup is None else max(3, args.warmup)
    res = run_cuda(args, cfg)
    if res is None:
        return
    if args.gpus == 1 and not args.no_cpu_baseline:
        n_tok, times, cores, sample = oracle_sample(cfg, steps=3, warmup=0)
        res["cpu_baseline"] = {"value": n_tok / float(np.min(times)), "unit": UNIT, "cores": cores,
                               "kind": "oracle", "sample": sample}
    print(json.dumps(res), flush=True)


if __name__ == "__main__":
    main()
