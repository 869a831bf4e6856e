#!/usr/bin/env python
"""Benchmark of the MoE feed-forward hot path on synthetic Llama-2-7B-shaped data.

    python bench.py --gpus 1 --steps 20 --warmup 5            # the CUDA path, one JSON line
    python bench.py --impl reference --steps 3 --warmup 1     # the CPU oracle on host cores
    python bench.py --workload fwd|decode|merge               # one of the other paths on its own

The headline is the training step (forward + backward) of one layer: T=16384 tokens, d_model 4096,
d_ff 11008, 4 experts, top-2, BF16 with FP32 accumulation.  On one GPU the same process then measures the
other configurations, one after the other with the previous one's buffers freed, and adds them to the
line under "sub": the forward alone at T=4096, the three routing variants at T=16384 (Switch top-1, soft
routing over all experts, top-2 with a skewed router), the decode-shaped forward over 32 layers and the
merge of four Llama-2-7B-shaped parameter sets, each with its own clock samples.

Under torchrun every rank runs an independent replica on its own batch (the path has no exchange
step), times K steps between barriers, and rank 0 prints whole-job tokens/s from the max time.
"""
from __future__ import annotations

import argparse
import gc
import hashlib
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

D_MODEL, D_FF, N_EXPERTS = 4096, 11008, 4
WORKLOADS = {
    # name: (T, k, seed, routing name, skewed router bias, forward+backward, layers)
    "fwd_bwd": (16384, 2, 2, "topk", False, True, 1),
    "fwd": (4096, 2, 1, "topk", False, False, 1),
    "switch_top1": (16384, 1, 3, "switch", False, True, 1),
    "soft_all4": (16384, 4, 3, "soft", False, True, 1),
    "top2_skewed": (16384, 2, 3, "topk", True, True, 1),
    "decode": (32, 2, 4, "topk", False, False, 32),
}
ALPHA = 0.01
SOAK_S = 2.0             # untimed run of the same step before the warm-up: power state and clocks settle
E2E_STEPS = 50

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of the seven tensor-core GEMM launches of one training
# step at T=16384, from the one-pass ncu capture summarised in profiles/tc_gemm_kernel_fwd_bwd_T16384_dram.txt
# (the traffic does not grow in proportion to T, so the T=4096 capture is not scaled).  The figure belongs to the
# kernel sources whose hash is recorded with it; with any other sources the bench reports traffic = null.
TC_GEMM_TRAFFIC = {"bytes_per_step_T16384": 33.68e9, "sources_sha256_16": "4b5584b3b2e0e287"}
TC_GEMM_SOURCES = ("btx_gemm_tc.cu", "btx_tc_ptx.cuh", "btx_common.cuh")
# The same for one launch (one layer) of the one-kernel decode-shaped forward, from the capture summarised in
# profiles/tc_small_forward_kernel_decode_T32_full.txt (1.0864 GB read + 0.0070 GB written).
SMALL_FWD_TRAFFIC = {"bytes_per_layer_T32": 1.0934e9, "sources_sha256_16": "59f3acb607798dbb"}
SMALL_FWD_SOURCES = ("btx_gemm_fused.cu", "btx_tc_ptx.cuh", "btx_route_dev.cuh", "btx_common.cuh")
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


def kernel_sources_hash(names=TC_GEMM_SOURCES):
    h = hashlib.sha256()
    for name in names:
        with open(os.path.join(ROOT, "paper_2403_07816_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


class ClockSampler:
    """Samples SM clocks, board power and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.proc = None
        self.gpu = gpu_index

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
        sm, mx, watts, reasons = [], [], [], set()
        for line in out.strip().splitlines():
            parts = [s.strip() for s in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            try:
                watts.append(float(parts[2]))
            except ValueError:
                pass
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm),
                "power_w": statistics.median(watts) if watts else None}


# ----------------------------------------------------------------------------------------------
# CPU oracle arm
# ----------------------------------------------------------------------------------------------

def oracle_step_fn(workload, tokens, device="cpu"):
    """Returns (fn, n_tokens): fn() runs the oracle (forward + backward for the training workloads) on the
    first `tokens` tokens of the workload's batch with the full expert weights."""
    import torch
    from oracle import btx_oracle as o
    from paper_2403_07816_b200 import synth
    T, k, seed, _, _, train, _ = WORKLOADS[workload]
    inp = synth.moe_inputs(T, D_MODEL, D_FF, N_EXPERTS, seed, torch.bfloat16, device)
    n = min(tokens, T)
    cpu = {name: synth.to_f64_numpy(t[:n] if name in ("x", "dy") else t) for name, t in inp.items()}

    def fn():
        o.moe_forward(cpu["x"], cpu["w_router"], cpu["w1"], cpu["w3"], cpu["w2"], k, alpha=ALPHA)
        if train:
            o.moe_backward(cpu["x"], cpu["w_router"], cpu["w1"], cpu["w3"], cpu["w2"], cpu["dy"], k, alpha=ALPHA)
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
    T, k = WORKLOADS[workload][0], WORKLOADS[workload][1]
    # A step of the oracle costs a fixed part (every expert's fp64 weights pass through the cores once, whatever
    # the batch) plus a part per token that grows a little faster than linearly.  Two calibration passes give
    # both; the sample is sized, with a safety factor and a cap of 4096 tokens, so that steps + warm-up take
    # about two and a half minutes, and one trial step at that size shrinks it further if it still runs long.
    def timed(n_tok):
        f, _ = oracle_step_fn(workload, n_tok)
        t0 = time.perf_counter(); f(); return time.perf_counter() - t0
    c_lo, c_hi = timed(64), timed(512)
    per_token = 1.5 * max((c_hi - c_lo) / 448.0, 1e-5)
    fixed = max(c_lo - 64 * per_token / 1.5, 0.0)
    total = args.steps + args.warmup + 1                 # + the trial step
    budget = 140.0 / total
    tokens = int((budget - fixed) / per_token) if budget > fixed else 16
    tokens = max(16, min(T, 4096, tokens // 16 * 16))
    fn, n = oracle_step_fn(workload, tokens)
    t0 = time.perf_counter(); fn(); trial = time.perf_counter() - t0
    if trial > 1.3 * budget and tokens > 16:
        tokens = max(16, int(tokens * budget / trial * 0.9) // 16 * 16)
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
        "config": {"workload": f"{workload}: first {n} of T={T} tokens per step, d_model={D_MODEL}, d_ff={D_FF}, "
                               f"E={N_EXPERTS}, top-{k}, fp64 CPU oracle (numpy/OpenBLAS)"},
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


def free_device_memory():
    import torch
    gc.collect()
    torch.cuda.empty_cache()


# kernels launched per call (memsets and copies are not counted)
LAUNCHES_FWD = 8          # router (its last block finalises the loss), 3 permutation kernels, gather, GEMM-1, GEMM-2, combine
LAUNCHES_FWD_SMALL = 6    # one-launch routing, gather, pass 1, SwiGLU fix-up, pass 2, combine
LAUNCHES_FWD_DENSE = 1    # inference with at most 64 tokens: the whole layer is one cooperative kernel
LAUNCHES_BWD = 11         # dy gather, dgrad-2, dgrad-1, 3 weight gradients, row-sum, dz, dW_l partial, dx combine, reduce


class MoeRun:
    """One configuration of the layer resident on the device: inputs, buffers and the step function."""

    def __init__(self, workload, dev, rank, tokens=0, layers=0):
        import torch
        from paper_2403_07816_b200 import binding as B, synth
        self.B, self.torch, self.dev = B, torch, dev
        T, k, seed, routing, skew, train, n_layers = WORKLOADS[workload]
        self.T = tokens or T
        self.k, self.train, self.workload = k, train, workload
        self.layers = layers or n_layers
        self.routing = {"topk": B.ROUTE_TOPK, "switch": B.ROUTE_SWITCH, "soft": B.ROUTE_SOFT}[routing]
        self.k_eff = N_EXPERTS if self.routing == B.ROUTE_SOFT else k
        d, F, E = D_MODEL, D_FF, N_EXPERTS
        # one independent seeded layer per decode "layer"; replicas differ by rank through the seed
        self.sets = [synth.moe_inputs(self.T, d, F, E, seed + 1000 * rank, torch.bfloat16, dev, layer=l, with_dy=train)
                     for l in range(self.layers)]
        self.bias = synth.skew_bias(E, dev) if skew else None
        self.desc = B.make_desc(self.T, d, F, E, k, torch.bfloat16, self.routing, ALPHA, False, train)
        self.ws, self.saved = B.alloc_buffers(self.desc, dev)
        self.y = torch.empty(self.T, d, dtype=torch.bfloat16, device=dev)
        self.routing_out = None
        if train:
            f32 = dict(dtype=torch.float32, device=dev)
            self.dx = torch.empty_like(self.y)
            self.dwr, self.dbias = torch.empty(E, d, **f32), torch.empty(E, **f32)
            self.dw1, self.dw3, self.dw2 = torch.empty(E, F, d, **f32), torch.empty(E, F, d, **f32), torch.empty(E, d, F, **f32)

    def forward(self, inp, routing_out=None):
        self.B.btx_moe_forward(self.desc, inp["x"], inp["w_router"], self.bias, inp["w1"], inp["w3"], inp["w2"], self.y,
                               routing_out, self.saved if self.train else None, self.ws)

    def backward(self, inp):
        self.B.btx_moe_backward(self.desc, inp["x"], inp["w_router"], self.bias, inp["w1"], inp["w3"], inp["w2"],
                                inp["dy"], 1.0, self.saved, self.dx, self.dwr, self.dbias, self.dw1, self.dw3, self.dw2,
                                0, self.ws)

    def step(self):
        for inp in self.sets:
            self.forward(inp)
            if self.train:
                self.backward(inp)

    def launches_per_step(self):
        fwd = LAUNCHES_FWD_SMALL if self.T * self.k_eff <= 1024 else LAUNCHES_FWD
        if not self.train and self.T <= 64:
            fwd = LAUNCHES_FWD_DENSE
        return (fwd + (LAUNCHES_BWD if self.train else 0)) * self.layers

    def flops_per_step(self, rows):
        return (18 if self.train else 6) * rows * D_MODEL * D_FF * self.layers

    def expert_counts(self):
        r = self.B.Routing.empty(self.desc, self.dev)
        self.forward(self.sets[0], r)
        self.torch.cuda.synchronize()
        return [int(v) for v in r.counts.cpu().tolist()]


def new_events(torch, n):
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
    for e in evs:
        e.record()                       # creates the handles the stage hook records into
    return evs


STAGES_F = ["route_permute_gather", "gemm1_swiglu", "gemm2_scatter", "combine"]
STAGES_B = ["gather_dy", "dgrad2_swiglu_bwd", "dgrad1", "wgrad_w2", "wgrad_w1", "wgrad_w3", "router_bwd"]


def soak(run, seconds):
    """Runs the step untimed for at least `seconds` (host clock, synchronising every few steps)."""
    torch = run.torch
    t0 = time.perf_counter()
    n = 0
    while True:
        for _ in range(4):
            run.step()
        n += 4
        torch.cuda.synchronize()
        if time.perf_counter() - t0 >= seconds:
            return time.perf_counter() - t0, n


def time_moe(run, K, W, world, local, soak_s, with_stages):
    """Soak, W warm-up steps, then exactly K timed steps between barriers with CUDA events on the launching
    stream and clock samples taken meanwhile.  Returns (ms per step, clocks, stage times or None, soak seconds)."""
    torch, B = run.torch, run.B
    soaked = 0.0
    if soak_s > 0:
        soaked, _ = soak(run, soak_s)
    for _ in range(W):
        run.step()
    torch.cuda.synchronize()
    assert B.btx_device_status(run.ws) == B.BTX_OK
    stage_events = None
    if with_stages and run.layers == 1:
        stage_events = [(new_events(torch, 5), new_events(torch, 8)) for _ in range(K)]
    sampler = ClockSampler(local)
    barrier(world)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(K):
        if stage_events is None:
            run.step()
            continue
        inp = run.sets[0]
        B.btx_set_stage_events(stage_events[i][0])
        run.forward(inp)
        if run.train:
            B.btx_set_stage_events(stage_events[i][1])
            run.backward(inp)
    B.btx_set_stage_events(None)
    e1.record()
    barrier(world)
    clocks = sampler.stop()
    ms = max_over_ranks(e0.elapsed_time(e1) / K, world, run.dev)
    assert B.btx_device_status(run.ws) == B.BTX_OK
    stages = None
    if stage_events is not None:
        stages = {}
        for i, nme in enumerate(STAGES_F):
            stages["fwd." + nme] = statistics.mean(se[0][i].elapsed_time(se[0][i + 1]) for se in stage_events)
        if run.train:
            for i, nme in enumerate(STAGES_B):
                stages["bwd." + nme] = statistics.mean(se[1][i].elapsed_time(se[1][i + 1]) for se in stage_events)
    return ms, clocks, stages, soaked


def tensor_roofline(run, rows, stages, clocks, timed_s, peaks):
    gemm_keys = [kname for kname in stages if "gemm" in kname or "grad" in kname]
    gemm_ms = sum(stages[kname] for kname in gemm_keys)
    achieved = run.flops_per_step(rows) / (gemm_ms * 1e-3) / 1e12
    # the sustained cuBLAS figure is the yardstick once the power cap has pulled the clocks down (or the
    # run, soak included, is long enough that it would have); a short un-capped run is compared with the burst figure
    sustained = "sw_power_cap" in (clocks.get("reasons") or []) or timed_s >= 1.0
    peak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
    traffic = None
    if (run.workload, run.T) == ("fwd_bwd", 16384) and kernel_sources_hash() == TC_GEMM_TRAFFIC["sources_sha256_16"]:
        traffic = TC_GEMM_TRAFFIC["bytes_per_step_T16384"]
    return {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
            "traffic": traffic, "peak_source": peaks["_source"] + (" sustained" if sustained else " burst"),
            "kernel": f"tc_gemm_kernel, {len(gemm_keys)} launches per step (flops of all / summed time)",
            "frac_of_nominal_2250": achieved / 2250.0}


def measure_e2e(run, world, steps):
    """The training step through the host-buffer entry point: pinned x, dy in; y, dx and the loss out, every step.
    Two steps are in flight, each on its own stream pair and buffer set (the weights are shared), so that the
    upload of step i+1 travels while step i computes: the way a training loop that keeps the GPU busy would call
    the entry point."""
    torch, B, dev = run.torch, run.B, run.dev
    inp = run.sets[0]
    hx = inp["x"].cpu().pin_memory(); hdy = inp["dy"].cpu().pin_memory()
    main = torch.cuda.current_stream(dev)
    lanes = []
    for i in range(2):
        ln = dict(stream=torch.cuda.Stream(device=dev), copy=torch.cuda.Stream(device=dev),
                  hy=torch.empty_like(hx).pin_memory(), hdx=torch.empty_like(hx).pin_memory(),
                  hloss=torch.empty(1, dtype=torch.float32).pin_memory(),
                  xd=torch.empty_like(inp["x"]), dyd=torch.empty_like(inp["x"]))
        if i == 0:
            ln.update(y=run.y, dx=run.dx, saved=run.saved, ws=run.ws, dwr=run.dwr, dbias=run.dbias, dw1=run.dw1,
                      dw3=run.dw3, dw2=run.dw2)
        else:
            ws2, saved2 = B.alloc_buffers(run.desc, dev)
            ln.update(y=torch.empty_like(run.y), dx=torch.empty_like(run.dx), saved=saved2, ws=ws2,
                      dwr=torch.empty_like(run.dwr), dbias=torch.empty_like(run.dbias), dw1=torch.empty_like(run.dw1),
                      dw3=torch.empty_like(run.dw3), dw2=torch.empty_like(run.dw2))
        lanes.append(ln)

    def e2e_step(i):
        ln = lanes[i % 2]
        with torch.cuda.stream(ln["stream"]):
            B.btx_moe_step_host(run.desc, hx, hdy, ln["hy"], ln["hdx"], ln["hloss"], ln["xd"], ln["dyd"], ln["y"],
                                ln["dx"], inp["w_router"], run.bias, inp["w1"], inp["w3"], inp["w2"], 1.0, ln["dwr"],
                                ln["dbias"], ln["dw1"], ln["dw3"], ln["dw2"], 0, ln["saved"], ln["ws"],
                                copy_stream=ln["copy"])

    def join():
        for ln in lanes:
            main.wait_stream(ln["stream"])

    def fork():
        for ln in lanes:
            ln["stream"].wait_stream(main)
    fork()
    for i in range(4):
        e2e_step(i)
    join()
    sampler = ClockSampler(dev.index or 0)
    barrier(world)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    fork()
    for i in range(steps):
        e2e_step(i)
    join()
    e1.record()
    barrier(world)
    clocks = sampler.stop()
    for ln in lanes:
        assert B.btx_device_status(ln["ws"]) == B.BTX_OK
    ems = max_over_ranks(e0.elapsed_time(e1) / steps, world, dev)
    act = run.T * D_MODEL * 2
    return {"value": run.T / (ems * 1e-3) * world, "unit": "tokens/s", "h2d_bytes_per_step": 2 * act,
            "d2h_bytes_per_step": 2 * act + 4, "ms_per_step": ems, "steps": steps, "clocks": clocks,
            "call": "btx_moe_step_host (pinned host x, dy in; y, dx, loss out), two steps in flight on two "
                    "stream pairs"}


def describe(run):
    T, k = run.T, run.k_eff
    if run.workload == "decode":
        return (f"decode: T={T} tokens x {run.layers} independent layers, d_model={D_MODEL}, d_ff={D_FF}, "
                f"E={N_EXPERTS}, top-{k}, bf16; {run.layers} distinct weight sets "
                f"({run.layers * 3 * N_EXPERTS * D_MODEL * D_FF * 2 / 1e9:.1f} GB) exceed L2")
    how = {"topk": f"top-{k}", "switch": "Switch top-1", "soft": f"soft routing over all {N_EXPERTS}"}[WORKLOADS[run.workload][3]]
    if run.bias is not None:
        how += ", router bias on expert 0 (first choice of about 70 % of the tokens)"
    return (f"{run.workload}: T={T} tokens, d_model={D_MODEL}, d_ff={D_FF}, E={N_EXPERTS}, {how}, bf16 with fp32 "
            f"accumulation, lb alpha {ALPHA}, {'forward+backward' if run.train else 'forward only'}; inputs (1.2 GB of "
            "weights and activations per step) exceed the 126 MB L2, no explicit flush")


def moe_result(run, ms, clocks, stages, soaked, K, W, world, peaks, with_counts):
    """Result object of one MoE configuration (used for the headline and for the sub-results)."""
    counts = run.expert_counts() if with_counts else None
    rows = sum(counts) if counts is not None else run.T * run.k_eff
    res = {"steps": K, "warmup": W, "soak_s": round(soaked, 2), "ms_per_step": ms, "clocks": clocks,
           "gpu_launches": run.launches_per_step() * K, "config": {"workload": describe(run)}}
    if counts is not None:
        res["expert_counts"] = counts
    if run.workload == "decode":
        w_bytes = run.layers * 3 * N_EXPERTS * D_MODEL * D_FF * 2
        gbs = w_bytes / (ms * 1e-3) / 1e9
        traffic = None                       # per launch = per layer, like `achieved`
        if run.T == 32 and kernel_sources_hash(SMALL_FWD_SOURCES) == SMALL_FWD_TRAFFIC["sources_sha256_16"]:
            traffic = SMALL_FWD_TRAFFIC["bytes_per_layer_T32"]
        res.update(metric="moe_ffn_decode_weight_stream_GBps", value=gbs * world, unit="GB/s",
                   roofline={"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                             "frac": gbs / peaks["hbm_gbs"], "frac_of_nominal_8000": gbs / 8000.0, "traffic": traffic,
                             "peak_source": peaks["_source"],
                             "kernel": "tc_small_forward_kernel (one launch per layer) over the whole step"})
    else:
        res.update(metric="moe_ffn_%s_tokens_per_s" % run.workload, value=run.T / (ms * 1e-3) * world, unit="tokens/s",
                   tflops=run.flops_per_step(rows) / (ms * 1e-3) / 1e12 * world)
        res["tflops_frac_of_nominal_2250"] = res["tflops"] / world / 2250.0
    if stages is not None:
        res["stages_ms"] = {kname: round(v, 4) for kname, v in stages.items()}
        if run.workload != "decode":
            res["roofline"] = tensor_roofline(run, rows, stages, clocks, soaked + ms * K * 1e-3, peaks)
    return res


def decode_stage_times(run):
    """Per-layer time of the decode path from one extra, untimed pass with an event before and after every layer
    (the layer is one kernel, so there are no stages inside it to time)."""
    torch, B = run.torch, run.B
    evs = [new_events(torch, 5) for _ in run.sets]
    for inp, ev in zip(run.sets, evs):
        B.btx_set_stage_events(ev)
        run.forward(inp)
    B.btx_set_stage_events(None)
    torch.cuda.synchronize()
    return {"fwd.layer": statistics.mean(ev[0].elapsed_time(ev[4]) for ev in evs)}


def run_moe(args, workload):
    import torch
    from paper_2403_07816_b200 import build as builder
    world, rank, local = dist_setup(args)
    if rank == 0:
        builder.build()
    barrier(world)
    dev = torch.device("cuda", local)
    peaks = load_peaks()
    K, W = args.steps, max(args.warmup, 3)
    soak_s = 0.0 if args.tokens or args.layers else args.soak_s    # profiler captures run few launches

    run = MoeRun(workload, dev, rank, tokens=args.tokens, layers=args.layers)
    ms, clocks, stages, soaked = time_moe(run, K, W, world, local, soak_s, with_stages=True)
    if workload == "decode":
        stages = decode_stage_times(run)
    line = {"n_gpus": world, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic"}
    line.update(moe_result(run, ms, clocks, stages, soaked, K, W, world, peaks, with_counts=False))
    line["e2e"] = measure_e2e(run, world, E2E_STEPS) if (run.train and not args.no_e2e) else None

    # ---- the other measured paths, one after the other (single GPU, default workload only) ----
    solo = rank == 0 and world == 1 and not args.tokens and not args.layers
    if solo and workload == "fwd_bwd" and not args.no_sub:
        sub = {}
        del run
        free_device_memory()
        for name in ("fwd", "switch_top1", "soft_all4", "top2_skewed", "decode"):
            r = MoeRun(name, dev, rank)
            k_sub = {"fwd": 200, "decode": 100}.get(name, 20)
            s_ms, s_clocks, s_stages, s_soaked = time_moe(r, k_sub, 3, 1, local, 1.0 if name in ("fwd", "decode") else SOAK_S,
                                                          with_stages=True)
            if name == "decode":
                s_stages = decode_stage_times(r)
            sub[name] = moe_result(r, s_ms, s_clocks, s_stages, s_soaked, k_sub, 3, 1, peaks, with_counts=True)
            del r
            free_device_memory()
        sub["merge"] = measure_merge(args, dev, local, 1, 20, 3, peaks)
        free_device_memory()
        line["sub"] = sub

    # ---- CPU oracle beside it (rank 0, single GPU only) ----
    if solo and not args.no_cpu_baseline and workload != "decode":
        free_device_memory()
        n_tok = 4096                           # about 10-30 s of host work
        fn, n = oracle_step_fn(workload, n_tok, device="cpu")
        t0 = time.perf_counter(); fn(); dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": n / dt, "unit": "tokens/s", "cores": host_cores(), "kind": "oracle",
                                "sample": f"first {n} of {WORKLOADS[workload][0]} tokens, full expert weights, one pass "
                                          f"({dt:.1f} s)"}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def measure_merge(args, dev, local, world, K, W, peaks):
    """btx_merge of four Llama-2-7B-shaped parameter sets, as many layers as fit (--merge-layers)."""
    import torch
    from paper_2403_07816_b200 import binding as B, synth
    n_models, d, F, vocab = 4, D_MODEL, D_FF, 32000
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
    return {"metric": "btx_merge_GBps", "value": gbs * world, "unit": "GB/s", "steps": K, "warmup": W,
            "ms_per_step": ms, "clocks": clocks, "gpu_launches": K,
            "config": {"workload": f"merge: 4 Llama-2-7B-shaped parameter sets, {layers} of 32 layers + embeddings/head "
                                   f"({read / 1e9:.1f} GB read, {written / 1e9:.1f} GB written per step, far beyond L2)"},
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "frac_of_nominal_8000": gbs / 8000.0, "traffic": None,
                         "peak_source": peaks["_source"], "kernel": "merge_kernel"}}


def run_merge(args):
    import torch
    from paper_2403_07816_b200 import build as builder
    world, rank, local = dist_setup(args)
    if rank == 0:
        builder.build()
    barrier(world)
    dev = torch.device("cuda", local)
    res = measure_merge(args, dev, local, world, args.steps, max(args.warmup, 3), load_peaks())
    line = {"n_gpus": world, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic", "e2e": None}
    line.update(res)
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0, help="timed steps (default 20; 100 for the short decode and merge steps)")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="btx", choices=["btx", "reference"])
    ap.add_argument("--workload", default="fwd_bwd", choices=list(WORKLOADS) + ["merge"])
    ap.add_argument("--merge-layers", type=int, default=32)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-sub", action="store_true", help="headline only: skip the other configurations")
    ap.add_argument("--soak-s", type=float, default=SOAK_S, help="untimed run of the step before the warm-up, seconds")
    ap.add_argument("--layers", type=int, default=0, help="decode: number of layers (profiling only)")
    ap.add_argument("--tokens", type=int, default=0, help="override T (profiling only; not a bench number)")
    args = ap.parse_args()
    if args.steps <= 0:     # steps of a few ms need more repetitions for the clock sampler to see the timed region
        short = {"decode": 100, "merge": 20, "fwd": 200}
        args.steps = short.get(args.workload, 20) if args.impl != "reference" else 20
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "merge":
        run_merge(args)
    else:
        run_moe(args, args.workload)


if __name__ == "__main__":
    main()
