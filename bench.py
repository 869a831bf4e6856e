#!/usr/bin/env python
"""Benchmark of the MoE feed-forward hot path (forward + backward) on synthetic Llama-2-7B-shaped
data: T=16384 tokens, d_model 4096, d_ff 11008, 4 experts, top-2, BF16 with FP32 accumulation.

    python bench.py --gpus 1 --steps 20 --warmup 5            # the CUDA path, one JSON line
    python bench.py --impl reference --steps 3 --warmup 1     # the CPU oracle on host cores
    python bench.py --workload fwd|decode|merge               # the other measured paths

Under torchrun every rank runs an independent replica on its own batch (the path has no exchange
step), times K steps between barriers, and rank 0 prints whole-job tokens/s from the max time.
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

WORKLOADS = {
    # name: (T, d_model, d_ff, E, k, seed)
    "fwd_bwd": (16384, 4096, 11008, 4, 2, 2),
    "fwd": (4096, 4096, 11008, 4, 2, 1),
    "decode": (32, 4096, 11008, 4, 2, 4),
}
ALPHA = 0.01
# dram__bytes_read.sum + dram__bytes_write.sum of the seven tc_gemm_kernel launches of one training step
# at T=16384 (26.38 GB read + 7.43 GB written); the algorithmic minimum is 10.3 GB read + 7.6 GB written
TC_GEMM_DRAM_BYTES_PER_STEP = 33.81e9
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.proc = None
        self.gpu = gpu_index
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        for line in out.strip().splitlines():
            parts = [s.strip() for s in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------------------------
# CPU oracle arm
# ----------------------------------------------------------------------------------------------

def oracle_step_fn(workload, tokens, device="cpu"):
    """Returns (fn, n_tokens): fn() runs the oracle forward + backward on the first `tokens` tokens
    of the workload's batch with the full expert weights."""
    import numpy as np
    import torch
    from oracle import btx_oracle as o
    from paper_2403_07816_b200 import synth
    T, d, F, E, k, seed = WORKLOADS[workload]
    inp = synth.moe_inputs(T, d, F, E, seed, torch.bfloat16, device)
    n = min(tokens, T)
    cpu = {name: synth.to_f64_numpy(t[:n] if name in ("x", "dy") else t) for name, t in inp.items()}

    def fn():
        if workload == "fwd_bwd":
            o.moe_forward(cpu["x"], cpu["w_router"], cpu["w1"], cpu["w3"], cpu["w2"], k, alpha=ALPHA)
            o.moe_backward(cpu["x"], cpu["w_router"], cpu["w1"], cpu["w3"], cpu["w2"], cpu["dy"], k, alpha=ALPHA)
        else:
            o.moe_forward(cpu["x"], cpu["w_router"], cpu["w1"], cpu["w3"], cpu["w2"], k, alpha=ALPHA)
    return fn, n


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    workload = args.workload if args.workload in ("fwd_bwd", "fwd") else "fwd_bwd"
    T, d, F, E, k, seed = WORKLOADS[workload]
    # size the sample so that steps+warmup fit in about two minutes: calibrate on 16 tokens
    fn, n = oracle_step_fn(workload, 16)
    t0 = time.perf_counter(); fn(); cal = time.perf_counter() - t0
    total = max(1, args.steps + args.warmup)
    budget = 120.0 / total
    tokens = int(max(16, min(T, 16 * budget / max(cal, 1e-3) * 0.6)))
    tokens = max(16, tokens // 16 * 16)
    fn, n = oracle_step_fn(workload, tokens)
    for _ in range(args.warmup):
        fn()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        fn()
    dt = (time.perf_counter() - t0) / max(1, args.steps)
    value = n / dt
    cores = host_cores()
    line = {
        "impl": "reference", "metric": "moe_ffn_%s_tokens_per_s" % workload, "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{workload}: first {n} of T={T} tokens per step, d_model={d}, d_ff={F}, E={E}, top-{k}, "
                               "fp64 CPU oracle (numpy/OpenBLAS)"},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                         "sample": f"{n} tokens per step, full expert weights"},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------
# CUDA arm
# ----------------------------------------------------------------------------------------------

def dist_setup(args):
    import torch
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    return world, rank, local


def barrier(world):
    import torch
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    if torch.cuda.is_available():
        torch.cuda.synchronize()


def max_over_ranks(value, world, device):
    import torch
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank, ms_local, world, device):
    """Whole-job units/s of N independent replicas: every rank processed `units_per_rank` in its own
    `ms_local`; the job took the slowest rank's time."""
    ms = max_over_ranks(ms_local, world, device)
    return units_per_rank * world / (ms * 1e-3), ms


def run_moe(args, workload):
    import torch
    from paper_2403_07816_b200 import binding as B, build as builder, synth
    world, rank, local = dist_setup(args)
    if rank == 0:
        builder.build()
    barrier(world)
    dev = torch.device("cuda", local)
    T, d, F, E, k, seed = WORKLOADS[workload]
    if args.tokens:
        T = args.tokens                      # reduced batch for profiler captures
    train = workload == "fwd_bwd"
    layers = (args.layers or 32) if workload == "decode" else 1
    K, W = args.steps, max(args.warmup, 3)
    peaks = load_peaks()

    # one independent seeded layer per decode "layer"; replicas differ by rank through the seed
    sets = [synth.moe_inputs(T, d, F, E, seed + 1000 * rank, torch.bfloat16, dev, layer=l, with_dy=train)
            for l in range(layers)]
    desc = B.make_desc(T, d, F, E, k, torch.bfloat16, B.ROUTE_TOPK, ALPHA, False, train)
    ws, saved = B.alloc_buffers(desc, dev)
    y = torch.empty(T, d, dtype=torch.bfloat16, device=dev)
    if train:
        f32 = dict(dtype=torch.float32, device=dev)
        dx = torch.empty_like(y)
        dwr, dbias = torch.empty(E, d, **f32), torch.empty(E, **f32)
        dw1, dw3, dw2 = torch.empty(E, F, d, **f32), torch.empty(E, F, d, **f32), torch.empty(E, d, F, **f32)

    def step(i=0):
        for inp in sets:
            B.btx_moe_forward(desc, inp["x"], inp["w_router"], None, inp["w1"], inp["w3"], inp["w2"], y, None,
                              saved if train else None, ws)
            if train:
                B.btx_moe_backward(desc, inp["x"], inp["w_router"], None, inp["w1"], inp["w3"], inp["w2"], inp["dy"],
                                   1.0, saved, dx, dwr, dbias, dw1, dw3, dw2, 0, ws)

    def new_events(n):
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
        for e in evs:
            e.record()                       # creates the handles the stage hook records into
        return evs

    for _ in range(W):
        step()
    torch.cuda.synchronize()
    assert B.btx_device_status(ws) == B.BTX_OK

    # ---- timed region: K steps between barriers, CUDA events on the launching stream ----
    stage_events = [(new_events(5), new_events(8)) for _ in range(K)] if layers == 1 else None
    sampler = ClockSampler(local)
    barrier(world)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(K):
        if stage_events is None:
            step()
            continue
        inp = sets[0]
        B.btx_set_stage_events(stage_events[i][0])
        B.btx_moe_forward(desc, inp["x"], inp["w_router"], None, inp["w1"], inp["w3"], inp["w2"], y, None,
                          saved if train else None, ws)
        if train:
            B.btx_set_stage_events(stage_events[i][1])
            B.btx_moe_backward(desc, inp["x"], inp["w_router"], None, inp["w1"], inp["w3"], inp["w2"], inp["dy"], 1.0,
                               saved, dx, dwr, dbias, dw1, dw3, dw2, 0, ws)
    B.btx_set_stage_events(None)
    e1.record()
    barrier(world)
    clocks = sampler.stop()
    ms = max_over_ranks(e0.elapsed_time(e1) / K, world, dev)
    assert B.btx_device_status(ws) == B.BTX_OK

    R = T * k
    flops_step = (18 if train else 6) * R * d * F * layers
    fwd_launches = 6 if T * k <= 1024 else 9        # small batches: routing+permutation in one launch, two passes + fix-up
    launches_per_step = (fwd_launches + (11 if train else 0)) * layers
    line = {
        "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "clocks": clocks,
        "gpu_launches": launches_per_step * K,
    }
    if workload == "decode":
        w_bytes = layers * 3 * E * d * F * 2
        gbs = w_bytes / (ms * 1e-3) / 1e9
        line.update(metric="moe_ffn_decode_weight_stream_GBps", value=gbs * world, unit="GB/s",
                    config={"workload": f"decode: T={T} tokens x {layers} independent layers, d_model={d}, d_ff={F}, "
                                        f"E={E}, top-{k}, bf16; {layers} distinct weight sets (34.6 GB) exceed L2"},
                    roofline={"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                              "frac": gbs / peaks["hbm_gbs"], "traffic": None, "peak_source": peaks["_source"],
                              "kernel": "tc_swapk_kernel (weight-streaming passes) over the whole step"})
        # per-layer stage times from one extra, untimed pass
        evs = [new_events(5) for _ in sets]
        for inp, ev in zip(sets, evs):
            B.btx_set_stage_events(ev)
            B.btx_moe_forward(desc, inp["x"], inp["w_router"], None, inp["w1"], inp["w3"], inp["w2"], y, None, None, ws)
        B.btx_set_stage_events(None)
        torch.cuda.synchronize()
        names_f = ["route_permute_gather", "gemm1_swiglu", "gemm2_scatter", "combine"]
        line["stages_ms"] = {"fwd." + nme: round(statistics.mean(ev[i].elapsed_time(ev[i + 1]) for ev in evs), 4)
                             for i, nme in enumerate(names_f)}
    else:
        tokens_s = T / (ms * 1e-3) * world
        line.update(metric="moe_ffn_%s_tokens_per_s" % workload, value=tokens_s, unit="tokens/s",
                    tflops=flops_step / (ms * 1e-3) / 1e12 * world,
                    config={"workload": f"{workload}: T={T} tokens, d_model={d}, d_ff={F}, E={E}, top-{k}, bf16 with "
                                        "fp32 accumulation, lb alpha 0.01; inputs (1.2 GB of weights and activations "
                                        "per step) exceed the 126 MB L2, no explicit flush"})
        # per-stage times averaged over the timed steps
        names_f = ["route_permute_gather", "gemm1_swiglu", "gemm2_scatter", "combine"]
        names_b = ["gather_dy", "dgrad2_swiglu_bwd", "dgrad1", "wgrad_w2", "wgrad_w1", "wgrad_w3", "router_bwd"]
        stages = {}
        for i, nme in enumerate(names_f):
            stages["fwd." + nme] = statistics.mean(se[0][i].elapsed_time(se[0][i + 1]) for se in stage_events)
        if train:
            for i, nme in enumerate(names_b):
                stages["bwd." + nme] = statistics.mean(se[1][i].elapsed_time(se[1][i + 1]) for se in stage_events)
        gemm_keys = [kname for kname in stages if "gemm" in kname or "grad" in kname]
        gemm_ms = sum(stages[kname] for kname in gemm_keys)
        achieved = flops_step / (gemm_ms * 1e-3) / 1e12
        # the sustained cuBLAS figure is the yardstick once the power cap has pulled the clocks down (or the
        # timed region is long enough that it would have); a short un-capped run is compared with the burst figure
        sustained = "sw_power_cap" in (clocks.get("reasons") or []) or ms * K >= 1000.0
        peak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
        line["stages_ms"] = {kname: round(v, 4) for kname, v in stages.items()}
        # DRAM bytes (read + write) of the seven launches of one step, from the ncu capture summarised in
        # profiles/tc_gemm_kernel_fwd_bwd_T16384_dram.txt; it holds for that workload only
        traffic = TC_GEMM_DRAM_BYTES_PER_STEP if (train and (T, d, F, E, k) == (16384, 4096, 11008, 4, 2)) else None
        line["roofline"] = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                            "frac": achieved / peak, "traffic": traffic, "peak_source": peaks["_source"] + (" sustained" if sustained else " burst"),
                            "kernel": f"tc_gemm_kernel, {len(gemm_keys)} launches per step (flops of all / summed time)",
                            "frac_of_nominal_2250": achieved / 2250.0}

    # ---- end to end through the host-buffer entry point (training workload only) ----
    if train and not args.no_e2e:
        # Two steps in flight, each on its own stream pair and buffer set (the weights are shared), so
        # that the upload of step i+1 travels while step i computes: the way a training loop that keeps
        # the GPU busy would call the entry point.  Every step still uploads its own x, dy and brings
        # back its own y, dx and loss inside the timed region.
        inp = sets[0]
        hx = inp["x"].cpu().pin_memory(); hdy = inp["dy"].cpu().pin_memory()
        Ke = max(4, min(K, 10))
        main = torch.cuda.current_stream(dev)
        lanes = []
        for i in range(2):
            ln = dict(stream=torch.cuda.Stream(device=dev), copy=torch.cuda.Stream(device=dev),
                      hy=torch.empty_like(hx).pin_memory(), hdx=torch.empty_like(hx).pin_memory(),
                      hloss=torch.empty(1, dtype=torch.float32).pin_memory(),
                      xd=torch.empty_like(inp["x"]), dyd=torch.empty_like(inp["x"]))
            if i == 0:
                ln.update(y=y, dx=dx, saved=saved, ws=ws, dwr=dwr, dbias=dbias, dw1=dw1, dw3=dw3, dw2=dw2)
            else:
                ws2, saved2 = B.alloc_buffers(desc, dev)
                ln.update(y=torch.empty_like(y), dx=torch.empty_like(dx), saved=saved2, ws=ws2,
                          dwr=torch.empty_like(dwr), dbias=torch.empty_like(dbias), dw1=torch.empty_like(dw1),
                          dw3=torch.empty_like(dw3), dw2=torch.empty_like(dw2))
            lanes.append(ln)

        def e2e_step(i):
            ln = lanes[i % 2]
            with torch.cuda.stream(ln["stream"]):
                B.btx_moe_step_host(desc, hx, hdy, ln["hy"], ln["hdx"], ln["hloss"], ln["xd"], ln["dyd"], ln["y"],
                                    ln["dx"], inp["w_router"], None, inp["w1"], inp["w3"], inp["w2"], 1.0, ln["dwr"],
                                    ln["dbias"], ln["dw1"], ln["dw3"], ln["dw2"], 0, ln["saved"], ln["ws"],
                                    copy_stream=ln["copy"])

        def join():
            for ln in lanes:
                main.wait_stream(ln["stream"])

        def fork():
            for ln in lanes:
                ln["stream"].wait_stream(main)
        fork()
        for i in range(2):
            e2e_step(i)
        join()
        barrier(world)
        e0.record()
        fork()
        for i in range(Ke):
            e2e_step(i)
        join()
        e1.record()
        barrier(world)
        for ln in lanes:
            assert B.btx_device_status(ln["ws"]) == B.BTX_OK
        ems = max_over_ranks(e0.elapsed_time(e1) / Ke, world, dev)
        act = T * d * 2
        line["e2e"] = {"value": T / (ems * 1e-3) * world, "unit": "tokens/s", "h2d_bytes_per_step": 2 * act,
                       "d2h_bytes_per_step": 2 * act + 4, "ms_per_step": ems, "steps": Ke,
                       "call": "btx_moe_step_host (pinned host x, dy in; y, dx, loss out), two steps in flight on two "
                               "stream pairs"}
    else:
        line["e2e"] = None

    # ---- CPU oracle beside it (rank 0, single GPU only) ----
    if rank == 0 and world == 1 and not args.no_cpu_baseline and workload != "decode" and not args.tokens:
        del sets
        torch.cuda.empty_cache()
        n_tok = 4096                           # about 10-30 s of host work
        fn, n = oracle_step_fn(workload, n_tok, device="cpu")
        t0 = time.perf_counter(); fn(); dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": n / dt, "unit": "tokens/s", "cores": host_cores(), "kind": "oracle",
                                "sample": f"first {n} of {T} tokens, full expert weights, one pass ({dt:.1f} s)"}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_merge(args):
    """btx_merge of four Llama-2-7B-shaped parameter sets, as many layers as fit (--merge-layers)."""
    import torch
    from paper_2403_07816_b200 import binding as B, build as builder, synth
    world, rank, local = dist_setup(args)
    if rank == 0:
        builder.build()
    barrier(world)
    dev = torch.device("cuda", local)
    peaks = load_peaks()
    n_models, d, F, vocab = 4, 4096, 11008, 32000
    layers = args.merge_layers
    free, _ = torch.cuda.mem_get_info(dev)
    per_layer = (4 * d * d + 2 * d + 3 * d * F) * 2
    embed = 2 * vocab * d * 2 + d * 2
    need = lambda L: (n_models * (L * per_layer + embed)) + (L * (4 * d * d + 2 * d) * 2 + embed + n_models * L * 3 * d * F * 2)
    while layers > 1 and need(layers) > 0.85 * free:
        layers -= 1
    shapes = synth.llama_like_param_shapes(layers, d, F, vocab)
    # sources: one big random buffer per model, carved into tensors (fast to generate)
    models, outputs = [], {}
    for m in range(n_models):
        total = 0
        for _, shp in shapes:
            n = 1
            for v in shp:
                n *= v
            total += n
        flat = torch.empty(total, dtype=torch.bfloat16, device=dev)
        chunk = 1 << 28                      # drawn in pieces so the fp32 staging stays small
        for ci, c0 in enumerate(range(0, total, chunk)):
            c1 = min(total, c0 + chunk)
            flat[c0:c1] = synth.normal((c1 - c0,), synth.WEIGHT_STD, 4, 100 + ci, torch.bfloat16, dev, layer=m)
        params, o = {}, 0
        for name, shp in shapes:
            n = 1
            for v in shp:
                n *= v
            params[name] = flat[o:o + n].view(shp)
            o += n
        models.append(params)
    for name, shp in shapes:
        outputs[name] = torch.empty(((n_models,) + tuple(shp)) if ".ffn." in name else tuple(shp),
                                    dtype=torch.bfloat16, device=dev)
    ws = torch.empty(B.btx_merge_workspace_size(n_models, len(shapes)), dtype=torch.uint8, device=dev)
    read = sum(models[0][n].numel() for n, _ in shapes) * 2 * n_models
    written = sum(t.numel() for t in outputs.values()) * 2
    K, W = args.steps, max(args.warmup, 3)
    for _ in range(W):
        B.btx_merge(models, outputs, ws)
    sampler = ClockSampler(local)
    barrier(world)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(K):
        B.btx_merge(models, outputs, ws)
    e1.record()
    barrier(world)
    clocks = sampler.stop()
    ms = max_over_ranks(e0.elapsed_time(e1) / K, world, dev)
    gbs = (read + written) / (ms * 1e-3) / 1e9
    line = {"metric": "btx_merge_GBps", "value": gbs * world, "unit": "GB/s", "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic", "clocks": clocks, "gpu_launches": K,
            "config": {"workload": f"merge: 4 Llama-2-7B-shaped parameter sets, {layers} of 32 layers + embeddings/head "
                                   f"({read / 1e9:.1f} GB read, {written / 1e9:.1f} GB written per step, far beyond L2)"},
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "traffic": None, "peak_source": peaks["_source"],
                         "kernel": "merge_kernel"},
            "e2e": None}
    if rank == 0:
        print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0, help="timed steps (default 20; 100 for the short decode and merge steps)")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="btx", choices=["btx", "reference"])
    ap.add_argument("--workload", default="fwd_bwd", choices=["fwd_bwd", "fwd", "decode", "merge"])
    ap.add_argument("--merge-layers", type=int, default=32)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--layers", type=int, default=0, help="decode: number of layers (profiling only)")
    ap.add_argument("--tokens", type=int, default=0, help="override T (profiling only; not a bench number)")
    args = ap.parse_args()
    if args.steps <= 0:     # steps of a few ms need more repetitions for the clock sampler to see the timed region
        short = {"decode": 100, "merge": 100, "fwd": 800}
        args.steps = short.get(args.workload, 20) if args.impl != "reference" else 20
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "merge":
        run_merge(args)
    else:
        run_moe(args, args.workload)


if __name__ == "__main__":
    main()
