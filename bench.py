#!/usr/bin/env python
"""Benchmark of the Bi-Mask layer step (mask + permutation search + three GEMMs).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

A "step" is one pass of the whole hot path (Alg. 1 body without the optimizer: forward mask and
pack, permutation search, backward mask and pack, sparse forward, sparse input gradient, dense
weight gradient) over every layer of the configuration; the metric is layer-steps per second.
One JSON line is printed by rank 0.  With N > 1 (torchrun) every rank runs an independent replica
(the step has no exchange between GPUs), and the value is the aggregate.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "bimask_layer_steps_per_sec"
UNIT = "layer-steps/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


# --------------------------------------------------------------------------------------------
# CPU oracle arm (reference / cpu_baseline)
# --------------------------------------------------------------------------------------------
ORACLE_PARTS = ("fwd_mask_pack", "candidates", "scoring", "bwd_mask_pack", "spmm_fwd", "spmm_dgrad", "wgrad")


def oracle_sample_time(cfg_id: int, rows: int = 1024, tokens: int = 256, cands: int = 4):
    """Times the CPU oracle, as it stands, on a bounded sample of every layer of the config (the first `rows` rows
    of W with the full input dim, `tokens` tokens, `cands` candidates), one timer per kind of step (the two mask
    passes, candidate generation, scoring, the three products), and scales each kind by its own work ratio to the
    full layer.  Returns (seconds for a full pass over all layers [extrapolated], seconds actually spent,
    description, per-kind record)."""
    from oracle import bimask_oracle as O
    from paper_2302_06058_b200 import inputs
    cfg = inputs.CONFIGS[cfg_id]
    total_full = 0.0
    spent = 0.0
    parts = {k: {"sample_s": 0.0, "full_s": 0.0} for k in ORACLE_PARTS}
    scales = []
    for li, L in enumerate(cfg.layers):
        Is, Ts, Ps = min(rows, L.I), min(tokens, L.T), min(cands, cfg.P)
        W = inputs.make_weight(Is, L.J, 1000 * cfg_id + 10 * li, cfg.init)
        X = inputs.make_activation(Ts, L.J, 1000 * cfg_id + 10 * li + 1)
        dY = inputs.make_activation(Ts, Is, 1000 * cfg_id + 10 * li + 2)
        t = [time.perf_counter()]
        B = O.forward_mask(W, cfg.N, cfg.M)
        O.forward_operand(W, B)
        t.append(time.perf_counter())
        cand = O.candidates(inputs.perm_seed(cfg_id), Ps, Is)
        t.append(time.perf_counter())
        _, perm, _ = O.perm_search(B, cand, cfg.N, cfg.M)
        t.append(time.perf_counter())
        Bbar = O.backward_mask(W, B, perm, cfg.N, cfg.M)
        Mb = O.unpermute_rows(Bbar, perm)
        O.backward_operand(W, Bbar, perm)
        t.append(time.perf_counter())
        O.spmm_fwd(X, W, B)
        t.append(time.perf_counter())
        O.spmm_dgrad(dY, W, Mb)
        t.append(time.perf_counter())
        O.wgrad(dY, X)
        t.append(time.perf_counter())
        r_mask = (L.I * L.J) / (Is * L.J)
        r_cand = (cfg.P * L.I) / (Ps * Is)
        r_score = (cfg.P * L.I * L.J) / (Ps * Is * L.J)
        r_gemm = (L.T * L.I * L.J) / (Ts * Is * L.J)
        ratio = dict(zip(ORACLE_PARTS, (r_mask, r_cand, r_score, r_mask, r_gemm, r_gemm, r_gemm)))
        for k, name in enumerate(ORACLE_PARTS):
            dt = t[k + 1] - t[k]
            parts[name]["sample_s"] += dt
            parts[name]["full_s"] += dt * ratio[name]
            total_full += dt * ratio[name]
        scales.append({"layer": li, "masks": r_mask, "candidates": r_cand, "scoring": r_score, "products": r_gemm})
        spent += t[-1] - t[0]
    desc = (f"config {cfg_id}: per layer the first {rows} rows of W (full input dim), {tokens} tokens, "
            f"{cands} candidates; every kind of step timed separately and scaled by its work ratio to the full "
            f"layer (extrapolated)")
    extrapolated = any(abs(v - 1.0) > 1e-9 for sc in scales for k, v in sc.items() if k != "layer")
    return total_full, spent, desc, {"parts": parts, "scale_factors": scales, "extrapolated": extrapolated}


def cpu_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
        return int(n)
    except Exception:
        return len(os.sched_getaffinity(0))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2302_06058_b200 import inputs
    cfg = inputs.CONFIGS[args.config]
    for _ in range(args.warmup):
        oracle_sample_time(args.config, rows=128, tokens=32, cands=1)
    # Size the per-step sample so that the whole run stays within a few minutes whatever --steps and the host are:
    # a time budget for the run, each step's sample sized from what the previous one cost (cost grows faster
    # than linearly in the rows, hence the margin); every step's result is scaled to the full layer anyway.
    budget = 150.0
    t_cal = time.perf_counter()
    oracle_sample_time(args.config, rows=128, tokens=args.ref_tokens, cands=2)
    last_rows, last_cost = 128, time.perf_counter() - t_cal
    per_pass = []
    rows_used = []
    t_begin = time.perf_counter()
    for k in range(args.steps):
        share = max(budget - (time.perf_counter() - t_begin), 0.0) / (args.steps - k)
        rows = int(last_rows * (share / max(last_cost, 1e-3)) ** 0.75) // 32 * 32
        rows = max(128, min(args.ref_rows, rows))
        t0 = time.perf_counter()
        full, _, desc, detail = oracle_sample_time(args.config, rows=rows, tokens=args.ref_tokens, cands=2)
        last_rows, last_cost = rows, time.perf_counter() - t0
        per_pass.append(full)
        rows_used.append(rows)
    if len(set(rows_used)) > 1:
        desc += f"; rows per step adapted to a {budget:.0f} s budget: {min(rows_used)}..{max(rows_used)}"
    wall = time.perf_counter() - t_begin
    sec = float(np.mean(per_pass))
    value = len(cfg.layers) / sec
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"config {args.config} ({cfg.name})", "layers": [[L.I, L.J, L.T] for L in cfg.layers],
                   "N": cfg.N, "M": cfg.M, "P": cfg.P},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": desc,
                         "extrapolated": detail["extrapolated"], "scale_factors": detail["scale_factors"],
                         "parts_last_step": detail["parts"]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0, "wall_s": wall,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------
# clocks sampler
# --------------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.gpu_id = gpu_id
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", self.gpu_id, f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        """Stop sampling (the samples stay on disk for window())."""
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.proc = None

    def close(self):
        try:
            os.unlink(self.path)
        except Exception:
            pass

    def window(self, t_begin=None, t_end=None):
        """Summary of the samples whose timestamp lies in [t_begin, t_end] (time.time())."""
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "power_w": None, "reasons": [], "samples": 0}
        if self.path is None:
            return out
        sm, mx, pw, reasons = [], [], [], set()
        try:
            with open(self.path) as f:
                for line in f:
                    p = [x.strip() for x in line.split(",")]
                    if len(p) < 8:
                        continue
                    try:
                        ts = datetime.datetime.strptime(p[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                        clk, cmax, watts = float(p[1]), float(p[2]), float(p[3])
                    except ValueError:
                        continue
                    if t_begin is not None and not (t_begin <= ts <= t_end):
                        continue
                    sm.append(clk)
                    mx.append(cmax)
                    pw.append(watts)
                    for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[4:8]):
                        if v.lower().startswith("active"):
                            reasons.add(name)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), power_w=float(np.median(pw)),
                       reasons=sorted(reasons), samples=len(sm))
        return out


# --------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------
# DRAM traffic per call (dram__bytes_read.sum + dram__bytes_write.sum over the kernels of the call, one ncu capture
# of `bench.py --profile` per layer of config 5); the capture is named in the JSON line beside the numbers.
NCU_TRAFFIC_SOURCE = "profiles/cfg5_launch_list.md"
NCU_TRAFFIC_BYTES = {
    (5, 0, "fwd_mask"): 268e6 + 64e6, (5, 1, "fwd_mask"): 269e6 + 69e6,
    (5, 0, "spmm_fwd"): 360e6 + 235e6, (5, 1, "spmm_fwd"): 592e6 + 51e6,
    (5, 0, "perm_search"): 17e6, (5, 1, "perm_search"): 11e6,              # generator + count kernel
    (5, 0, "bwd_mask"): 277e6 + 62e6, (5, 1, "bwd_mask"): 277e6 + 61e6,
    (5, 0, "spmm_dgrad"): 269e6 + 216e6 + 592e6 + 51e6,                    # permute pass + product
    (5, 1, "spmm_dgrad"): 67e6 + 19e6 + 365e6 + 236e6,
    (5, 0, "wgrad"): 1402e6 + 249e6, (5, 1, "wgrad"): 1117e6 + 249e6,
}


def job_value(world: int, n_layers: int, steps: int, ms_max_over_ranks: float) -> float:
    """Whole-job throughput of N independent replicas: every rank runs `steps` passes over `n_layers` layers, the
    job takes as long as its slowest rank."""
    return world * n_layers * steps / (ms_max_over_ranks * 1e-3)


def max_over_ranks(values, world: int, device="cpu"):
    """Element-wise maximum of a list of per-rank timings over all ranks (the only collective of the bench)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def clock_regime(clocks: dict, timed_region_s=None) -> str:
    """"burst": the sampled SM clock (median) stayed near its maximum, and the timed region, when given, was too short
    for the power cap to bite; "sustained" otherwise.  Decides which measured tensor peak a fraction is quoted
    against."""
    near_max = bool(clocks.get("sm_mhz")) and bool(clocks.get("sm_max_mhz")) and clocks["sm_mhz"] >= 0.9 * clocks["sm_max_mhz"]
    if near_max and (timed_region_s is None or timed_region_s < 1.0):
        return "burst"
    return "sustained"


def algorithmic_work(L, P):
    """Algorithmic bytes / flops per launch of each timed call for one layer."""
    I, J, T = L.I, L.J, L.T
    IJ = I * J
    return {
        "fwd_mask": {"bound": "hbm", "bytes": 4 * IJ + IJ + IJ / 8 + IJ / 8 + 2 * IJ / 8},
        # quoted against one HBM pass over W; the mask bits it really reads (P * IJ / 8 bytes) come out of L2
        "perm_search": {"bound": "hbm", "bytes": 4 * IJ, "l2_bytes": P * IJ / 8},
        "bwd_mask": {"bound": "hbm", "bytes": 4 * IJ + IJ / 8 + 4 * I + IJ + IJ / 8 + IJ / 8 + 2 * IJ / 8},
        "spmm_fwd": {"bound": "tensor", "flops": 2.0 * T * IJ, "bytes": 2 * T * J + 1.125 * IJ + 2 * T * I},
        "spmm_dgrad": {"bound": "tensor", "flops": 2.0 * T * IJ, "bytes": 2 * T * I + 1.125 * IJ + 2 * T * J + 4 * T * I},
        "wgrad": {"bound": "tensor", "flops": 2.0 * T * IJ, "bytes": 2 * T * I + 2 * T * J + 4 * IJ},
    }


def run_gpu(args):
    import torch
    import torch.distributed as dist
    import paper_2302_06058_b200 as bm
    from paper_2302_06058_b200 import inputs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    cfg = inputs.CONFIGS[args.config]
    seed = inputs.perm_seed(args.config)
    peaks = load_peaks()
    stream = torch.cuda.current_stream()

    layers = []
    host = []
    for li, L in enumerate(cfg.layers):
        if args.profile and li != args.layer:
            continue
        W, X, dY = inputs.make_layer(args.config, li)
        b = bm.alloc_layer_buffers(L.T, L.I, L.J, cfg.P)
        hW = torch.from_numpy(W).pin_memory()
        hX = torch.from_numpy(X.view(np.int16)).view(torch.bfloat16).pin_memory()
        hdY = torch.from_numpy(dY.view(np.int16)).view(torch.bfloat16).pin_memory()
        b["W"], b["X"], b["dY"] = hW.cuda(), hX.cuda(), hdY.cuda()
        largs = bm.make_layer_args(L.T, L.I, L.J, cfg.N, cfg.M, cfg.P, seed, True, b)
        layers.append((L, b, largs))
        host.append({"W": hW, "X": hX, "dY": hdY})
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    if args.profile:
        # one layer, the individual C-ABI calls in step order: the command line used under ncu
        L, b, largs = layers[0]
        wsb = b["ws"].numel()
        for _ in range(args.warmup + args.steps):
            bm.bimask_fwd_mask(b["W"], L.I, L.J, cfg.N, cfg.M, b["maskbits_f"], b["vals_f"], b["meta_f"], b["hw_meta_f"])
            bm.bimask_spmm_fwd(b["X"], b["vals_f"], b["hw_meta_f"], L.T, L.I, L.J, b["Y"], b["status_word"])
            bm.bimask_perm_search(b["maskbits_f"], L.I, L.J, cfg.N, cfg.M, cfg.P, seed, None, b["perm"], b["best_idx"],
                                  b["counts"], b["ws"], wsb)
            bm.bimask_bwd_mask(b["W"], b["maskbits_f"], b["perm"], L.I, L.J, cfg.N, cfg.M, b["maskbits_b"], b["vals_b"],
                               b["meta_b"], b["hw_meta_b"])
            bm.bimask_spmm_dgrad(b["dY"], b["perm"], b["vals_b"], b["hw_meta_b"], L.T, L.I, L.J, b["dX"], b["ws"], wsb,
                                 b["status_word"])
            bm.bimask_wgrad(b["dY"], b["X"], L.T, L.I, L.J, b["dW"], b["ws"], wsb, b["status_word"])
            torch.cuda.synchronize()
        print(json.dumps({"profile": True, "config": args.config, "layer": args.layer,
                          "status": int(b["status_word"].item())}), flush=True)
        return

    def one_step():
        for _, _, largs in layers:
            bm.bimask_layer_step(largs)

    graph = None
    launches_per_step = None
    if args.graph:
        # capture one pass over all layers in a CUDA graph and replay it: removes the host-side
        # launch cost, which dominates the small configurations
        one_step()                                        # first calls set kernel attributes: not capturable
        torch.cuda.synchronize()
        cap_stream = torch.cuda.Stream()
        cap_stream.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        n0 = bm.bimask_launch_count()
        with torch.cuda.graph(graph, stream=cap_stream):
            for _, _, largs in layers:
                largs.stream = torch.cuda.current_stream().cuda_stream
                bm.bimask_layer_step(largs)
        launches_per_step = bm.bimask_launch_count() - n0
        for _, _, largs in layers:
            largs.stream = stream.cuda_stream
        step_fn = graph.replay
    else:
        step_fn = one_step

    # ---- warm-up, then the timed region: K steps through bimask_layer_step ----
    gpu_uuid = str(local)
    try:
        gpu_uuid = "GPU-" + str(torch.cuda.get_device_properties(local).uuid)
    except Exception:
        pass
    sampler = ClockSampler(gpu_uuid)
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        step_fn()
    barrier()
    launches0 = bm.bimask_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_head_begin = time.time()
    ev0.record(stream)
    for _ in range(args.steps):
        step_fn()
    ev1.record(stream)
    barrier()
    t_head_end = time.time()
    step_ms_total = ev0.elapsed_time(ev1)
    launches = bm.bimask_launch_count() - launches0
    if graph is not None:
        launches = launches_per_step * args.steps          # replayed from the graph, counted at capture

    # ---- the same step with the search switched off (the permutation of the last search is kept):
    #      Algorithm 1 searches once per Delta T = 100 iterations, so this is the common iteration.
    #      Reported beside the headline, never as it.
    nosearch = [bm.make_layer_args(L.T, L.I, L.J, cfg.N, cfg.M, cfg.P, seed, False, b) for L, b, _ in layers]
    for a in nosearch:
        bm.bimask_layer_step(a)
    barrier()
    en0, en1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    en0.record(stream)
    for _ in range(args.steps):
        for a in nosearch:
            bm.bimask_layer_step(a)
    en1.record(stream)
    barrier()
    nosearch_ms_total = en0.elapsed_time(en1)

    # ---- per-call breakdown over the same K steps (CUDA events between the C-ABI calls) ----
    names = ["fwd_mask", "spmm_fwd", "perm_search", "bwd_mask", "spmm_dgrad", "wgrad"]
    acc = {li: {n: 0.0 for n in names} for li in range(len(layers))}
    time.sleep(1.0)      # an idle second: the breakdown starts from the same power state as the headline's timed region
    t_call_begin = time.time()
    all_evs = []
    for _ in range(args.steps):
        evs = []
        for li, (L, b, _) in enumerate(layers):
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(7)]
            wsb = b["ws"].numel()
            ev[0].record(stream)
            bm.bimask_fwd_mask(b["W"], L.I, L.J, cfg.N, cfg.M, b["maskbits_f"], b["vals_f"], b["meta_f"], b["hw_meta_f"])
            ev[1].record(stream)
            bm.bimask_spmm_fwd(b["X"], b["vals_f"], b["hw_meta_f"], L.T, L.I, L.J, b["Y"], b["status_word"])
            ev[2].record(stream)
            bm.bimask_perm_search(b["maskbits_f"], L.I, L.J, cfg.N, cfg.M, cfg.P, seed, None, b["perm"], b["best_idx"],
                                  b["counts"], b["ws"], wsb)
            ev[3].record(stream)
            bm.bimask_bwd_mask(b["W"], b["maskbits_f"], b["perm"], L.I, L.J, cfg.N, cfg.M, b["maskbits_b"], b["vals_b"],
                               b["meta_b"], b["hw_meta_b"])
            ev[4].record(stream)
            bm.bimask_spmm_dgrad(b["dY"], b["perm"], b["vals_b"], b["hw_meta_b"], L.T, L.I, L.J, b["dX"], b["ws"], wsb,
                                 b["status_word"])
            ev[5].record(stream)
            bm.bimask_wgrad(b["dY"], b["X"], L.T, L.I, L.J, b["dW"], b["ws"], wsb, b["status_word"])
            ev[6].record(stream)
            evs.append(ev)
        all_evs.append(evs)
    torch.cuda.synchronize()      # once, after the last pass: every call follows the one before it as in the timed step
    t_call_end = time.time()
    # per call the MEDIAN over the passes, times the number of passes (the first call after the idle second starts on an
    # idle GPU and would carry its launch latency into a mean)
    for li in range(len(layers)):
        for k, n in enumerate(names):
            per_pass = sorted(evs[li][k].elapsed_time(evs[li][k + 1]) for evs in all_evs)
            acc[li][n] = per_pass[len(per_pass) // 2] * args.steps

    # ---- the same step repeated back to back for --sustain-s seconds: the figure under the power cap ----
    sustain_ms, sustain_steps, t_sus_begin, t_sus_end = 0.0, 0, None, None
    if args.sustain_s > 0:
        batch = max(1, int(0.25 / max(step_ms_total / args.steps * 1e-3, 1e-6)))      # about 0.25 s per batch
        t_sus_begin = time.time()
        batches = []
        while time.time() - t_sus_begin < args.sustain_s:
            es0, es1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            es0.record(stream)
            for _ in range(batch):
                step_fn()
            es1.record(stream)
            es1.synchronize()
            batches.append(es0.elapsed_time(es1))
        barrier()
        t_sus_end = time.time()
        tail = batches[len(batches) // 2:]                  # the second half: the clocks have settled
        sustain_ms, sustain_steps = float(sum(tail)), batch * len(tail)

    sampler.stop()
    clocks = sampler.window(t_head_begin, t_head_end)     # samples taken inside the headline's timed region
    clocks_calls = sampler.window(t_call_begin, t_call_end)
    clocks_sustain = sampler.window(t_sus_begin + 0.5 * (t_sus_end - t_sus_begin), t_sus_end) if t_sus_begin else None
    if not clocks["samples"]:                             # a timed region shorter than the sampling period
        clocks = sampler.window(t_head_begin - 0.05, t_head_end + 0.05)
    sampler.close()
    status = [int(b["status_word"].item()) for _, b, _ in layers]
    if any(status):
        raise RuntimeError(f"device status words non-zero: {status}")

    # ---- roofline of every call, and of the dominant one.  A tensor-bound call is quoted against both measured
    #      peaks (burst: a kernel timed alone at full clock; sustained: inside a long run under the power cap) and
    #      `frac` is the one that matches the clocks sampled while the calls were timed. ----
    regime = clock_regime(clocks, step_ms_total * 1e-3)
    # (a per-call loop too short for the sampler to catch takes the regime of the timed run just before it)
    regime_calls = clock_regime(clocks_calls) if clocks_calls.get("samples") else regime
    kernels = []
    for li, (L, b, _) in enumerate(layers):
        work = algorithmic_work(L, cfg.P)
        for n in names:
            ms = acc[li][n] / args.steps
            w = work[n]
            entry = {"layer": li, "call": n, "ms": ms}
            if w["bound"] == "hbm":
                entry.update(bound="hbm", achieved=w["bytes"] / (ms * 1e-3) / 1e9, peak=peaks["hbm_gbs"], unit="GB/s")
                entry["frac"] = entry["achieved"] / entry["peak"]
                if "l2_bytes" in w:
                    # what the count kernel really moves: mask bits out of L2, against the rate at which 148 SMs can
                    # take data from L2 (64 bytes per clock each) at the sampled clock
                    mhz = clocks_calls.get("sm_mhz") or clocks_calls.get("sm_max_mhz") or 1965.0
                    entry["l2_tbs"] = w["l2_bytes"] / (ms * 1e-3) / 1e12
                    entry["l2_fill_peak_tbs"] = 148 * 64 * mhz * 1e6 / 1e12
                    entry["l2_frac"] = entry["l2_tbs"] / entry["l2_fill_peak_tbs"]
            else:
                mult = 1.0 if n == "wgrad" else 2.0       # the 2:4 products: nominal sparse : dense ratio
                entry.update(bound="tensor", achieved=w["flops"] / (ms * 1e-3) / 1e12, unit="TFLOP/s",
                             peak_burst=mult * peaks["bf16_tflops"], peak_sustained=mult * peaks["bf16_tflops_sustained"])
                entry["frac_burst"] = entry["achieved"] / entry["peak_burst"]
                entry["frac_sustained"] = entry["achieved"] / entry["peak_sustained"]
                entry["peak"] = entry["peak_burst"] if regime_calls == "burst" else entry["peak_sustained"]
                entry["frac"] = entry["achieved"] / entry["peak"]
            t = NCU_TRAFFIC_BYTES.get((args.config, li, n))
            if t is not None:
                entry["traffic"] = t
                entry["algorithmic_bytes"] = w["bytes"]
            kernels.append(entry)
    dom = max(kernels, key=lambda e: e["ms"])
    roofline = {"bound": dom["bound"], "achieved": dom["achieved"], "peak": dom["peak"], "unit": dom["unit"],
                "frac": dom["frac"], "traffic": dom.get("traffic"),
                "traffic_source": NCU_TRAFFIC_SOURCE if dom.get("traffic") is not None else None,
                "kernel": f"layer {dom['layer']} {dom['call']}", "regime": regime_calls,
                "peak_source": peaks["source"] + (f" ({regime_calls} bf16" + ("; x2 for the 2:4 sparse products)"
                                                                              if dom["call"] != "wgrad" else ")")
                                                   if dom["bound"] == "tensor" else " (copy bandwidth)")}
    if dom["bound"] == "tensor":
        roofline.update(frac_burst=dom["frac_burst"], frac_sustained=dom["frac_sustained"])
    if dom["frac"] > 1.05:
        roofline["note"] = "fraction above 1: the kernel ran at a higher clock than the peak measurement; see frac_burst"

    # ---- end to end through the host-buffer entry point ----
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    host_args = []
    h2d = d2h = 0
    for (L, b, largs), hb in zip(layers, host):
        ho = {"W": hb["W"], "X": hb["X"], "dY": hb["dY"],
              "Y": torch.empty(L.T, L.I, dtype=torch.bfloat16).pin_memory(),
              "dX": torch.empty(L.T, L.J, dtype=torch.bfloat16).pin_memory(),
              "dW": torch.empty(L.I, L.J, dtype=torch.float32).pin_memory(),
              "perm": torch.empty(L.I, dtype=torch.int32).pin_memory(),
              "best_idx": torch.empty(1, dtype=torch.int32).pin_memory(),
              "counts": torch.empty(cfg.P, dtype=torch.int64).pin_memory()}
        hst = torch.zeros(1, dtype=torch.int32).pin_memory()
        host_args.append((bm.make_layer_args(L.T, L.I, L.J, cfg.N, cfg.M, cfg.P, seed, True, ho), ho, hst))
        h2d += sum(hb[k].numel() * hb[k].element_size() for k in ("W", "X", "dY"))
        d2h += sum(ho[k].numel() * ho[k].element_size() for k in ("Y", "dX", "dW", "perm", "best_idx", "counts")) + 4
    for (L, b, largs), (ha, _, hst) in zip(layers, host_args):      # one untimed pass
        bm.bimask_layer_step_host(largs, ha, hst)
    # the copies share the host's PCIe and memory system with other tenants of the machine: two repetitions of the
    # timed region, the faster one is reported
    e2e_runs = []
    for _ in range(2):
        barrier()
        t0 = time.perf_counter()
        ee0, ee1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ee0.record(stream)
        for _ in range(e2e_steps):
            for (L, b, largs), (ha, _, hst) in zip(layers, host_args):
                bm.bimask_layer_step_host_async(largs, ha, hst)     # upload of one layer overlaps the download of the last
        bm.bimask_host_sync()
        ee1.record(stream)
        barrier()
        e2e_runs.append(max(ee0.elapsed_time(ee1), (time.perf_counter() - t0) * 1e3))
    e2e_ms = min(e2e_runs)

    # ---- whole iterations of Algorithm 1 (search every 100th call, SGD update fused with the next
    #      forward mask); runs last because it changes W in place.  Reported beside the headline. ----
    moms = [torch.zeros(L.I, L.J, dtype=torch.float32, device="cuda") for L, _, _ in layers]
    tstate = {"t": 1}

    def train_pass():
        for (L, b, largs), mom in zip(layers, moms):
            bm.bimask_train_step(bm.make_train_args(largs, mom, 1e-6, 0.9, 1e-4, tstate["t"], 100, tstate["t"] > 1))
        tstate["t"] += 1

    for _ in range(3):
        train_pass()
    barrier()
    et0, et1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    et0.record(stream)
    for _ in range(args.steps):
        train_pass()
    et1.record(stream)
    barrier()
    train_ms_total = et0.elapsed_time(et1)
    status = [int(b["status_word"].item()) for _, b, _ in layers]
    if any(status):
        raise RuntimeError(f"device status words non-zero after the training iterations: {status}")

    # ---- max over ranks ----
    step_ms_total, e2e_ms, nosearch_ms_total, train_ms_total, sustain_ms = max_over_ranks(
        [step_ms_total, e2e_ms, nosearch_ms_total, train_ms_total, sustain_ms], world, "cuda")
    nl = len(layers)
    value = job_value(world, nl, args.steps, step_ms_total)
    e2e_value = job_value(world, nl, e2e_steps, e2e_ms)

    if rank == 0:
        cpu_full, cpu_spent, desc, cpu_detail = oracle_sample_time(args.config, rows=args.ref_rows, tokens=args.ref_tokens,
                                                                   cands=2)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": step_ms_total / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"config {args.config} ({cfg.name})",
                       "layers": [[L.I, L.J, L.T] for L in cfg.layers], "N": cfg.N, "M": cfg.M, "P": cfg.P,
                       "search_every_step": True, "parallelism": f"replicas x{world}", "cuda_graph": bool(args.graph),
                       "l2": "inputs larger than L2 (W alone is %.0f MB per layer)" % (cfg.layers[0].I * cfg.layers[0].J * 4 / 1e6)
                       if cfg.layers[0].I * cfg.layers[0].J * 4 > 126e6 else "inputs smaller than L2: warm-cache numbers"},
            "clocks": clocks, "regime": regime, "clocks_per_call": clocks_calls,
            "sustained": ({"value": job_value(world, nl, sustain_steps, sustain_ms), "unit": UNIT,
                           "ms_per_step": sustain_ms / sustain_steps, "seconds": args.sustain_s, "steps": sustain_steps,
                           "clocks": clocks_sustain,
                           "note": "the same step back to back for --sustain-s seconds, second half of the run timed"}
                          if sustain_steps else None),
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps, "repetitions_ms": e2e_runs,
                    "api": "bimask_layer_step_host_async + bimask_host_sync (pinned host buffers)"},
            "gpu_launches": int(launches),
            "search_off": {"value": world * nl * args.steps / (nosearch_ms_total * 1e-3), "unit": UNIT,
                           "ms_per_step": nosearch_ms_total / args.steps,
                           "note": "do_search=0: permutation kept from the last search; not the headline",
                           "delta_t_100_value": world * nl * 100.0 /
                           ((99.0 * nosearch_ms_total + step_ms_total) / args.steps * 1e-3)},
            "train_step": {"value": world * nl * args.steps / (train_ms_total * 1e-3), "unit": UNIT,
                           "ms_per_step": train_ms_total / args.steps,
                           "note": "bimask_train_step: Algorithm 1 iterations t = 4.., search when t % 100 == 0, SGD "
                                   "(momentum, weight decay) fused with the next forward mask; not the headline"},
            "roofline": roofline,
            "kernels": kernels,
            "cpu_baseline": {"value": nl / cpu_full, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                             "sample": desc, "cpu_seconds_spent": cpu_spent, "extrapolated": cpu_detail["extrapolated"],
                             "scale_factors": cpu_detail["scale_factors"], "parts": cpu_detail["parts"]},
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_per_call(args):
    """Side measurement: every C-ABI call of the path alone, 5 warm-up + --steps timed launches each, CUDA events,
    min and median; "cold" = a 256 MB buffer is overwritten and a second one read before every launch (L2 flushed and
    left clean: after the write alone the timed kernel would also pay for the write-back of up to 126 MB of dirty
    lines, about 19 us; clocks near burst because of the gaps), "warm" = back to back.  Fractions are against the
    burst peaks (copy bandwidth, bf16 burst)."""
    import torch
    import paper_2302_06058_b200 as bm
    from paper_2302_06058_b200 import inputs
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    cfg = inputs.CONFIGS[args.config]
    seed = inputs.perm_seed(args.config)
    peaks = load_peaks()
    pN, pM = cfg.N, cfg.M
    if args.pattern:                                          # another N:M pattern on the same shapes, e.g. 4:8 or 2:8
        pN, pM = (int(v) for v in args.pattern.split(":"))
    pack = pN <= 2                                            # N > 2: dense masked operands, dense products
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    flush_rd = torch.zeros(64 << 20, dtype=torch.int32, device="cuda")
    reps = max(args.steps, 20) if args.steps != 100 else 20
    out = []
    for li, L in enumerate(cfg.layers):
        W, X, dY = inputs.make_layer(args.config, li)
        b = bm.alloc_layer_buffers(L.T, L.I, L.J, cfg.P, dense=not pack)
        b["W"] = torch.from_numpy(W).cuda()
        b["X"] = torch.from_numpy(X.view(np.int16)).cuda().view(torch.bfloat16)
        b["dY"] = torch.from_numpy(dY.view(np.int16)).cuda().view(torch.bfloat16)
        if not pack:
            b["meta_f"] = b["hw_meta_f"] = b["meta_b"] = b["hw_meta_b"] = None
        wsb = b["ws"].numel()
        mom = torch.zeros(L.I, L.J, device="cuda")
        calls = {
            "fwd_mask": lambda: bm.bimask_fwd_mask(b["W"], L.I, L.J, pN, pM, b["maskbits_f"], b["vals_f"], b["meta_f"],
                                                   b["hw_meta_f"]),
            "spmm_fwd": lambda: bm.bimask_spmm_fwd(b["X"], b["vals_f"], b["hw_meta_f"], L.T, L.I, L.J, b["Y"], b["status_word"]),
            "perm_search": lambda: bm.bimask_perm_search(b["maskbits_f"], L.I, L.J, pN, pM, cfg.P, seed, None, b["perm"],
                                                         b["best_idx"], b["counts"], b["ws"], wsb),
            "bwd_mask": lambda: bm.bimask_bwd_mask(b["W"], b["maskbits_f"], b["perm"], L.I, L.J, pN, pM, b["maskbits_b"],
                                                   b["vals_b"], b["meta_b"], b["hw_meta_b"]),
            "spmm_dgrad": lambda: bm.bimask_spmm_dgrad(b["dY"], b["perm"], b["vals_b"], b["hw_meta_b"], L.T, L.I, L.J, b["dX"],
                                                       b["ws"], wsb, b["status_word"]),
            "wgrad": lambda: bm.bimask_wgrad(b["dY"], b["X"], L.T, L.I, L.J, b["dW"], b["ws"], wsb, b["status_word"]),
            "sgd_fwd_mask": lambda: bm.bimask_sgd_fwd_mask(b["W"], b["dW"], mom, L.I, L.J, pN, pM, 1e-9, 0.9, 1e-4,
                                                           b["maskbits_f"], b["vals_f"], b["meta_f"], b["hw_meta_f"]),
            "layer_step": lambda: bm.bimask_layer_step(bm.make_layer_args(L.T, L.I, L.J, pN, pM, cfg.P, seed, True, b)),
        }
        work = algorithmic_work(L, cfg.P)
        work["sgd_fwd_mask"] = {"bound": "hbm", "bytes": 21.4 * L.I * L.J}
        work["layer_step"] = {"bound": "tensor", "flops": 6.0 * L.T * L.I * L.J}
        for name, fn in calls.items():
            res = {"layer": li, "call": name}
            for kind in ("cold", "warm"):
                for _ in range(5):
                    fn()
                torch.cuda.synchronize()
                ts = []
                for _ in range(reps):
                    if kind == "cold":
                        flush.zero_()
                        flush_rd.max()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    fn()
                    e1.record()
                    torch.cuda.synchronize()
                    ts.append(e0.elapsed_time(e1) * 1e3)
                res[kind + "_us_min"] = min(ts)
                res[kind + "_us_median"] = float(np.median(ts))
            w = work[name]
            t = res["cold_us_median"] * 1e-6
            if w["bound"] == "hbm":
                res.update(bound="hbm", achieved=w["bytes"] / t / 1e9, peak=peaks["hbm_gbs"], unit="GB/s")
            else:
                pk = peaks["bf16_tflops"] * (1.0 if (name in ("wgrad", "layer_step") or not pack) else 2.0)
                res.update(bound="tensor", achieved=w["flops"] / t / 1e12, peak=pk, unit="TFLOP/s")
            res["frac"] = res["achieved"] / res["peak"]
            out.append(res)
        if int(b["status_word"].item()):
            raise RuntimeError("device status word non-zero")
        del b
    print(json.dumps({"per_call": out, "config": args.config, "pattern": f"{pN}:{pM}", "launches_per_kind": reps,
                      "peak_source": peaks["source"],
                      "note": "fractions of the burst peaks from the cold median"}), flush=True)


# ResNet-50's 3x3 convolutions (H, W, C, I, stride): the stride-1 layers of the four stages, then the three down-sampling ones
CONV_LAYERS = [(56, 56, 64, 64, 1), (28, 28, 128, 128, 1), (14, 14, 256, 256, 1), (7, 7, 512, 512, 1),
               (56, 56, 128, 128, 2), (28, 28, 256, 256, 2), (14, 14, 512, 512, 2)]


def run_conv(args):
    """Side measurement, not the headline: the convolution form of the layer step (bimask_conv_layer_step) on
    ResNet-50's 3x3 layers at batch --conv-batch, explicit and automatic form, CUDA events per step."""
    import torch
    import paper_2302_06058_b200 as bm
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    N, M, P, NB = 2, 4, 100, args.conv_batch
    gen = torch.Generator(device="cuda").manual_seed(7)
    rows = []
    for (H, W, C, I, stride) in CONV_LAYERS:
        Ho, Wo = (H - 1) // stride + 1, (W - 1) // stride + 1
        T, J = NB * Ho * Wo, 9 * C
        b = bm.alloc_layer_buffers(T, I, J, P)
        b["W"] = torch.randn(I, J, device="cuda", generator=gen) * (2.0 / J) ** 0.5
        b["X"] = torch.randn(NB, H, W, C, device="cuda", generator=gen).bfloat16()
        b["dY"] = torch.randn(NB, Ho, Wo, I, device="cuda", generator=gen).bfloat16()
        b["dX"] = torch.empty(NB, H, W, C, dtype=torch.bfloat16, device="cuda")
        b["ws"] = torch.empty(bm.bimask_conv_workspace_bytes(NB, H, W, C, I, P, stride), dtype=torch.uint8, device="cuda")
        largs = bm.make_layer_args(T, I, J, N, M, P, 43, True, b)
        row = {"layer": [NB, H, W, C, I], "stride": stride}
        for name, mode in (("explicit", 1), ("auto", 0), ("implicit", 2)):
            ca = bm.make_conv_args(largs, NB, H, W, C, mode, stride)
            n0 = bm.bimask_launch_count()
            for _ in range(max(args.warmup, 3)):
                bm.bimask_conv_layer_step(ca)
            launches = (bm.bimask_launch_count() - n0) // max(args.warmup, 3)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(args.steps):
                bm.bimask_conv_layer_step(ca)
            e1.record()
            torch.cuda.synchronize()
            row[name] = {"us_per_step": e0.elapsed_time(e1) * 1e3 / args.steps, "launches": int(launches)}
        if int(b["status_word"].item()):
            raise RuntimeError("device status word non-zero")
        rows.append(row)
    print(json.dumps({"workload": "3x3 convolution layer steps (ResNet-50 shapes), 2:4, P = 100, search on",
                      "conv": rows, "steps": args.steps, "note": "inputs smaller than L2: warm-cache numbers"}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=5, help="workload: 1..5 (default 5, the largest)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--sustain-s", type=float, default=3.0,
                    help="also repeat the step back to back for this many seconds and report that figure (0: skip)")
    ap.add_argument("--graph", action="store_true", help="replay one captured pass (CUDA graph) in the timed region")
    ap.add_argument("--profile", action="store_true", help="run only the C-ABI calls of one layer (for ncu)")
    ap.add_argument("--layer", type=int, default=0)
    ap.add_argument("--ref-rows", type=int, default=1024)
    ap.add_argument("--ref-tokens", type=int, default=256)
    ap.add_argument("--per-call", action="store_true", help="time every C-ABI call alone (cold and warm L2, min and median)")
    ap.add_argument("--pattern", default=None, help="with --per-call: another N:M pattern on the config's shapes, e.g. 4:8")
    ap.add_argument("--conv", action="store_true", help="time the convolution form of the layer step instead")
    ap.add_argument("--conv-batch", type=int, default=32)
    args = ap.parse_args()
    if args.conv and args.impl != "reference":
        run_conv(args)
        return
    if args.per_call and args.impl != "reference":
        run_per_call(args)
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
