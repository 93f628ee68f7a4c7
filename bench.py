#!/usr/bin/env python
"""Throughput of the SliceMoE layer forward on B200, one JSON line per run.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg1] [--impl ours|reference] [--backward]

A step is one whole layer forward (route -> dispatch -> expert FFN -> combine) over one batch of
seeded synthetic tokens.  `value` is tokens/s with the inputs already in HBM, the K steps captured once
and replayed as one CUDA graph (`ms_per_step_plain_launches` is the same K steps launched one by one); `e2e` is the same
through slicemoe_forward_host with pinned host buffers (copies inside the timed region).  The
path does not shard: with --gpus N every rank runs an independent replica on its own batch
(weak scaling, no data-path collective) and `value` is the sum over ranks / max time.

With --backward the line gains a `backward` object: slicemoe_backward timed on the same batches (up to 10
steps; not part of `value`).  `--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

L2_BYTES = 126e6
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised in
# profiles/fused_forward_cfg1_cfg2.md and profiles/three_launch_forward_cfg1_cfg2.md (taken on cfg2,
# whose tokens exceed L2).  The other workloads of the same slice width scale it by the rows one launch
# processes (traffic is proportional to rows: every row is read once per chosen expert and written once).
NCU_TRAFFIC_CFG2 = {"route": 134.328064e6 + 142.558720e6, "dispatch": 17.735168e6 + 0.924928e6,
                    "expert_ffn": 451.720704e6 + 175.928320e6,
                    "fused_forward": 578.811136e6 + 352.389888e6}
NCU_TRAFFIC_ROWS_CFG2 = 65536 * 16
# dram__bytes_read + dram__bytes_write of the two backward kernels on cfg1 (profiles/backward_cfg1.md)
NCU_TRAFFIC_BACKWARD_CFG1 = (43.363072e6 + 26.524160e6) + (87.232256e6 + 5.461248e6)
NCU_TRAFFIC_ROWS_CFG1 = 16384 * 8


def ncu_traffic(stage, lc):
    if stage not in NCU_TRAFFIC_CFG2 or lc.ds != 64 or lc.k != 2:
        return None
    return NCU_TRAFFIC_CFG2[stage] * lc.N / NCU_TRAFFIC_ROWS_CFG2


# tanh.approx results per clock per SM (measured, profiles/microbenchmarks_b200.md): the GELU(tanh) experts
# cannot go faster than R_kept * F / (148 * 16) cycles, whatever the tensor pipe does.
TANH_PER_CLK_PER_SM = 16.0
N_SM = 148


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


# --------------------------------------------------------------------------------------------
# workload arithmetic: algorithmic FLOPs (router 2N(ds Hr + Hr E), experts 4 R_kept ds F) and compulsory bytes
# --------------------------------------------------------------------------------------------
def layer_work(lc, kept_rows, touched_experts):
    b = 2 if lc.dtype == "bf16" else 4
    ds = lc.ds
    router_flops = 2.0 * lc.N * (ds * lc.Hr + lc.Hr * lc.E)
    expert_flops = 4.0 * kept_rows * ds * lc.F
    io_bytes = 2.0 * lc.T * lc.d * b
    router_w = (lc.Hr * ds + lc.Hr + lc.E * lc.Hr + lc.E) * b
    expert_w = touched_experts * (2 * ds * lc.F + lc.F + ds) * b
    return dict(router_flops=router_flops, expert_flops=expert_flops,
                total_flops=router_flops + expert_flops,
                compulsory_bytes=io_bytes + router_w + expert_w,
                # per-stage algorithmic figures of the staged pipeline
                stage_flops=dict(route=router_flops, expert_ffn=expert_flops),
                stage_bytes=dict(
                    route=lc.T * lc.d * b + router_w + lc.R * 8,
                    dispatch=lc.R * 8 + lc.R * 8 + kept_rows * ds * b * 2,      # idx+p in, dest+perm out, row read+write
                    expert_ffn=2.0 * kept_rows * ds * b + expert_w,
                    combine=kept_rows * ds * b + lc.R * 4 + lc.T * lc.d * b))


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.samples = []
        self._stop = threading.Event()
        self._thread = None

    def _run(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}",
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True,
                                     timeout=5).stdout.strip()
                if out:
                    self.samples.append([x.strip() for x in out.split(",")])
            except Exception:
                pass
            self._stop.wait(0.1)

    def __enter__(self):
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._thread.join(timeout=10)

    def summary(self):
        mhz, mx, reasons = [], None, set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for s in self.samples:
            try:
                mhz.append(float(s[0]))
                mx = float(s[1])
                for name, v in zip(names, s[2:6]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                continue
        mhz.sort()
        return {"sm_mhz": mhz[len(mhz) // 2] if mhz else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(mhz)}


def shard_tokens(T_per_rank, world):
    """Replicas only: every rank processes its own batch of T tokens (weak scaling)."""
    return [T_per_rank] * world


def aggregate(tokens_per_rank_per_step, steps, seconds_per_rank):
    """Whole-job tokens/s: all ranks' tokens over the slowest rank's time."""
    return sum(tokens_per_rank_per_step) * steps / max(seconds_per_rank)


def max_over_ranks(times, dist=None, device="cpu"):
    """Element-wise maximum of a list of per-rank timings over all ranks (identity without a group)."""
    import torch
    t = torch.tensor(list(times), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


# --------------------------------------------------------------------------------------------
# CPU oracle leg (also the `--impl reference` arm)
# --------------------------------------------------------------------------------------------
def time_oracle(lc, target_s=12.0, steps=1, warmup=0):
    """Times oracle.forward on the first T_s tokens of the workload; T_s is sized from a short
    calibration run so that one call takes about target_s seconds."""
    import oracle
    from paper_2510_04286_b200 import synth
    probe_T = min(lc.T, 64)
    sub = lc.with_tokens(probe_T)
    h, w = synth.make_layer_inputs(sub)
    ocfg = oracle.OracleConfig(T=sub.T, d=sub.d, S=sub.S, E=sub.E, k=sub.k, Hr=sub.Hr, F=sub.F,
                               act=sub.act, capacity=sub.capacity)
    oracle.forward(ocfg, h, w)
    t0 = time.perf_counter()
    oracle.forward(ocfg, h, w)
    rate = probe_T / max(time.perf_counter() - t0, 1e-6)
    T_s = int(max(probe_T, min(lc.T, rate * target_s)))
    if steps == 1 and T_s == lc.T:
        # the whole workload takes less than the target: repeat it to reach about target_s of CPU work
        steps = int(max(1, min(64, round(target_s * rate / lc.T))))
    sub = lc.with_tokens(T_s)
    h, w = synth.make_layer_inputs(sub)
    ocfg = oracle.OracleConfig(T=sub.T, d=sub.d, S=sub.S, E=sub.E, k=sub.k, Hr=sub.Hr, F=sub.F,
                               act=sub.act, capacity=sub.capacity)
    for _ in range(warmup):
        oracle.forward(ocfg, h, w)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.forward(ocfg, h, w)
    dt = time.perf_counter() - t0
    return dict(value=T_s * steps / dt, unit="tokens/s", cores=oracle.threads(), kind="oracle",
                sample=f"first {T_s} of {lc.T} tokens of {lc.name}, {steps} call(s), fp64, OpenMP over rows",
                seconds=dt, tokens=T_s)


def run_reference(args, lc):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    per_call = max(0.5, min(12.0, 120.0 / (steps + warmup)))
    r = time_oracle(lc, target_s=per_call, steps=steps, warmup=warmup)
    line = {
        "impl": "reference", "metric": "SliceMoE layer fwd tokens/s", "value": r["value"],
        "unit": "tokens/s", "n_gpus": args.gpus, "steps": steps, "warmup": warmup,
        "ms_per_step": 1e3 * r["seconds"] / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(lc, sets=1),
        "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")},
        "e2e": {"value": r["value"], "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(lc, sets, wsets=1):
    l2 = (f"rotating {sets} distinct token/output buffer sets between steps (larger than the 126 MB L2)"
          if sets > 1 else "single buffer set")
    if wsets > 1:
        l2 += f" and {wsets} copies of the weights (token sets alone would fit in L2 beside them)"
    return {"workload": lc.name, "T": lc.T, "d": lc.d, "S": lc.S, "E": lc.E, "k": lc.k, "F": lc.F,
            "Hr": lc.Hr, "act": "gelu_tanh" if lc.act else "relu", "capacity": lc.capacity, "l2": l2}


# --------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------
def run_ours(args, lc):
    import numpy as np
    import torch
    import paper_2510_04286_b200 as sm
    from paper_2510_04286_b200 import synth, tensors

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    cfg = tensors.config_from_synth(lc)
    tdt = sm.torch_dtype(cfg)
    b = 2 if lc.dtype == "bf16" else 4
    set_bytes = 2 * lc.T * lc.d * b
    sets = int(max(2, min(64, -(-2.2 * L2_BYTES // set_bytes)))) if set_bytes < 2.2 * L2_BYTES else 2
    # distinct seeded batches: rank r, set s draws seed 1000*r + s
    w_np = synth.make_weights(lc)
    w = tensors.weights_to_torch(w_np, lc.dtype)
    # Small batches (decode) would leave everything L2-resident however many token sets rotate: the
    # weights, their largest input, rotate too until tokens + weights exceed 2.2 x L2.
    w_bytes = sum(int(t.numel()) * t.element_size() for t in w.values() if t is not None)
    short = 2.2 * L2_BYTES - sets * set_bytes
    wsets = int(max(1, min(16, -(-short // w_bytes)))) if short > 0 else 1
    w_all = [w] + [{n: (None if t is None else t.clone()) for n, t in w.items()} for _ in range(wsets - 1)]
    hs = [tensors.to_torch(synth.make_tokens(lc, seed=1000 * rank + s), lc.dtype) for s in range(sets)]
    outs = [torch.empty((lc.T, lc.d), dtype=tdt, device="cuda") for _ in range(sets)]
    ws = sm.alloc_workspace(cfg)
    assigned = torch.empty((lc.E,), dtype=torch.int32, device="cuda")
    kept = torch.empty((lc.E,), dtype=torch.int32, device="cuda")

    def step(i):
        sm.slicemoe_forward(cfg, w_all[i % wsets], hs[i % sets], outs[i % sets], ws, assigned, kept)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # The clock sampler (an nvidia-smi child every 100 ms) starts before the warm-up so that spawning
    # it does not compete with the launching thread inside the timed region; it keeps sampling through
    # all three timed regions below.
    clocks = ClockSampler(local)
    clocks.__enter__()
    warm = max(3, args.warmup)
    for i in range(warm):
        step(i)
    torch.cuda.synchronize()
    if sm.slicemoe_last_status(ws) != 0:
        raise RuntimeError(f"device status {sm.slicemoe_last_status(ws)} after warm-up")
    kept_rows = int(kept.sum().item())
    touched = int((kept > 0).sum().item())
    # routing balance of this batch (Eq. 2 with alpha = 0.1, Section 4's ELE), computed on the device
    stats = torch.empty(2, dtype=torch.float64, device="cuda")
    sm.slicemoe_load_stats(assigned, 0.1, stats)
    l_cap, ele = (float(x) for x in stats.cpu())

    # ---- timed region 1: device-resident inputs -------------------------------------------
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    launches0 = sm.slicemoe_launch_count()
    start.record()
    for i in range(args.steps):
        step(i)
    stop.record()
    barrier()
    launches = sm.slicemoe_launch_count() - launches0
    t_dev = start.elapsed_time(stop) / 1e3

    # the same steps on ONE buffer set (tokens, outputs and weights stay in L2 where they fit): reported
    # beside the rotating (cold) figure, never as `value`
    start.record()
    for i in range(args.steps):
        sm.slicemoe_forward(cfg, w, hs[0], outs[0], ws, assigned, kept)
    stop.record()
    barrier()
    t_warm = start.elapsed_time(stop) / 1e3

    # ---- timed region 2: host buffers through the C ABI -----------------------------------
    h_host = [tensors.to_torch(synth.make_tokens(lc, seed=1000 * rank + s), lc.dtype, "cpu", pin=True)
              for s in range(min(sets, 4))]
    o_host = [torch.empty_like(x).pin_memory() for x in h_host]
    for i in range(3):
        sm.slicemoe_forward_host(cfg, w, h_host[i % len(h_host)], o_host[i % len(h_host)], ws, assigned, kept)
    barrier()
    start.record()
    for i in range(args.steps):
        sm.slicemoe_forward_host(cfg, w, h_host[i % len(h_host)], o_host[i % len(h_host)], ws, assigned, kept)
    stop.record()
    barrier()
    t_e2e = start.elapsed_time(stop) / 1e3

    # ---- timed region 3: per-stage CUDA events (recorded by the library on its stream) ----
    # (the stage-timed call keeps one launch per stage; the forward timed above is one launch)
    ev = [sm.StageEvents() for _ in range(min(args.steps, 64))]
    for i in range(3):
        sm.slicemoe_forward_profiled(cfg, w, hs[i % sets], outs[i % sets], ws, ev[0], assigned, kept)
    barrier()
    for i in range(len(ev)):
        sm.slicemoe_forward_profiled(cfg, w_all[i % wsets], hs[i % sets], outs[i % sets], ws, ev[i], assigned, kept)
    torch.cuda.synchronize()
    stage_ms = np.mean([e.stage_ms() for e in ev], axis=0)

    # ---- timed region 4 (--backward): slicemoe_backward on the same batches -----------------
    # Not part of `value`: the headline metric is the forward, and the default run launches the forward's
    # kernels only.  Each set's expert ids and gates come
    # from its own forward; grad_out is a seeded N(0, 1) batch per set.
    bwd = None
    bws = None
    if args.backward:
        try:
            bws = torch.empty(sm.slicemoe_backward_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
        except sm.SliceMoEError:
            bws = None      # shape outside the backward kernels' tile set
    if bws is not None:
        idxs = [torch.empty((cfg.N, cfg.k), dtype=torch.int32, device="cuda") for _ in range(sets)]
        gates = [torch.empty((cfg.N, cfg.k), dtype=torch.float32, device="cuda") for _ in range(sets)]
        gouts = [tensors.to_torch(synth.make_grad_out(lc, seed=1000 * rank + s), lc.dtype) for s in range(sets)]
        for s_ in range(sets):
            sm.slicemoe_forward(cfg, w, hs[s_], outs[s_], ws, assigned, kept, idxs[s_], gates[s_])
        shapes = dict(dWr1=(cfg.Hr, cfg.ds), dbr1=(cfg.Hr,), dWr2=(cfg.E, cfg.Hr), dbr2=(cfg.E,),
                      dW1=(cfg.E, cfg.F, cfg.ds), db1=(cfg.E, cfg.F), dW2=(cfg.E, cfg.ds, cfg.F), db2=(cfg.E, cfg.ds))
        grads = {n: torch.empty(sh, dtype=torch.float32, device="cuda") for n, sh in shapes.items()}
        bsteps = max(1, min(args.steps, 10))

        def bstep(i):
            j = i % sets
            sm.slicemoe_backward(cfg, w, hs[j], gouts[j], idxs[j], gates[j], outs[j], grads, bws)

        for i in range(3):
            bstep(i)
        barrier()
        l0 = sm.slicemoe_launch_count()
        start.record()
        for i in range(bsteps):
            bstep(i)
        stop.record()
        barrier()
        bwd = dict(t=start.elapsed_time(stop) / 1e3 / bsteps, steps=bsteps,
                   launches_per_step=(sm.slicemoe_launch_count() - l0) // bsteps)
        (bwd["t"],) = max_over_ranks([bwd["t"]], dist, device="cuda")

    # ---- last region: the K steps of region 1 captured once and replayed as ONE CUDA graph -----
    # (one forward per node, same rotating buffers; the gaps between launches shrink.  This is the timing
    # behind `value`; region 1's plain launches are reported beside it and stand in if capture fails.
    # Last, so that a failed capture cannot disturb another region.)
    t_graph = None
    try:
        graph = torch.cuda.CUDAGraph()
        # thread-local capture mode: CUDA calls of other threads (a process group's watchdog) do not
        # invalidate the capture
        with torch.cuda.graph(graph, capture_error_mode="thread_local"):
            for i in range(args.steps):
                step(i)
        graph.replay()
        barrier()
        start.record()
        graph.replay()
        stop.record()
        barrier()
        t_graph = start.elapsed_time(stop) / 1e3
    except Exception as ex:          # capture is an extra: say why it is missing and go on
        sys.stderr.write(f"graph replay not measured: {ex}\n")
    clocks.__exit__(None, None, None)

    # `value` is the graph replay (one forward per graph node, rotating buffers) where every rank captured
    # it, else the plain launches of region 1
    t_dev, t_e2e, t_graph_max, graph_failed = max_over_ranks(
        [t_dev, t_e2e, t_graph or 0.0, 0.0 if t_graph else 1.0], dist, device="cuda")
    use_graph = graph_failed == 0.0
    t_plain = t_dev
    if use_graph:
        t_dev = t_graph_max

    if rank == 0:
        peaks, peak_src = load_peaks()
        work = layer_work(lc, kept_rows, touched)
        stages = dict(zip(sm.STAGES, (float(x) for x in stage_ms)))
        dom = max(stages, key=stages.get)
        t_step = t_dev / args.steps
        single_launch = launches == args.steps
        if single_launch:
            # the timed forward is ONE kernel (router, dispatch and expert phases): its launch
            # duration is the step time measured by the events around the timed region
            dom = "fused_forward"
            achieved = work["total_flops"] / t_step / 1e12
            roof = {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"}
            stages = dict(stages, fused_forward=1e3 * t_step)
        elif dom in work["stage_flops"]:
            achieved = work["stage_flops"][dom] / (stages[dom] * 1e-3) / 1e12
            roof = {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"}
        else:
            achieved = work["stage_bytes"][dom] / (stages[dom] * 1e-3) / 1e9
            roof = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
        roof.update(frac=roof["achieved"] / roof["peak"], traffic=ncu_traffic(dom, lc),
                    kernel=dom, kernel_ms=stages[dom], peak_source=f"of {peak_src}")
        t_tensor = work["total_flops"] / (peaks["bf16_tflops"] * 1e12)
        t_hbm = work["compulsory_bytes"] / (peaks["hbm_gbs"] * 1e9)
        line = {
            "metric": "SliceMoE layer fwd tokens/s", "value": aggregate(shard_tokens(lc.T, world), args.steps, [t_dev]),
            "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
            "ms_per_step": 1e3 * t_step, "timing": ("one CUDA graph of the K steps, replayed" if use_graph
                                                     else "K plain launches (graph capture failed)"),
            "ms_per_step_plain_launches": 1e3 * t_plain / args.steps,
            "ms_per_step_same_buffers": 1e3 * t_warm / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": lc.dtype, "data": "synthetic", "config": workload_config(lc, sets, wsets),
            "routed_slices_per_s": world * lc.R / t_step,
            "routing_stats": {"ele": ele, "l_cap_alpha_0.1": l_cap},
            "e2e": {"value": world * lc.T * args.steps / t_e2e, "unit": "tokens/s",
                    "h2d_bytes_per_step": lc.T * lc.d * b, "d2h_bytes_per_step": lc.T * lc.d * b},
            "gpu_launches": int(launches),
            "clocks": clocks.summary(),
            "roofline": roof,
            "stage_ms_one_launch_per_stage": {k: v for k, v in stages.items() if k != "fused_forward"},
            "activation_bound": {
                "what": "tanh unit: R_kept*F GELU(tanh) evaluations at 16 per clock per SM",
                "t_us": (1e6 * kept_rows * lc.F / (N_SM * TANH_PER_CLK_PER_SM) / (clocks.summary()["sm_max_mhz"] or 1965.0) / 1e6
                         if lc.act else 0.0)},
            "layer_roofline": {"t_tensor_us": 1e6 * t_tensor, "t_hbm_us": 1e6 * t_hbm,
                               "bound": "tensor" if t_tensor >= t_hbm else "hbm",
                               "frac": max(t_tensor, t_hbm) / t_step, "kept_rows": kept_rows,
                               "touched_experts": touched, "peak_source": f"of {peak_src}"},
        }
        if bwd is not None:
            # algorithmic work of a backward = twice the forward's (input and weight gradient of every
            # product); the kernels also redo the forward's products (recompute factor 1.5).  fp32 on
            # CUDA cores: the bound is the FMA pipes, 128 lanes x 2 FLOP per clock per SM.
            alu_peak = N_SM * 128 * 2 * (clocks.summary()["sm_max_mhz"] or 1965.0) * 1e6 / 1e12
            ach = 2.0 * work["total_flops"] / bwd["t"] / 1e12
            line["backward"] = {
                "ms_per_step": 1e3 * bwd["t"], "tokens_per_s": world * lc.T / bwd["t"], "steps": bwd["steps"],
                "gpu_launches_per_step": int(bwd["launches_per_step"]), "dtype": "f32",
                "roofline": {"bound": "alu", "achieved": ach, "peak": alu_peak, "unit": "TFLOP/s",
                             "frac": ach / alu_peak,
                             "traffic": (NCU_TRAFFIC_BACKWARD_CFG1 * lc.N / NCU_TRAFFIC_ROWS_CFG1
                                         if lc.ds == 64 and lc.k == 2 and lc.F == 256 else None),
                             "peak_source": "derived: 148 SMs x 128 fp32 lanes x 2 FLOP x max SM clock"}}
        if world == 1 and not args.no_cpu_baseline:
            r = time_oracle(lc)
            line["cpu_baseline"] = {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")}
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="cfg1")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--backward", action="store_true",
                    help="also time slicemoe_backward on the same batches (the `backward` object of the line)")
    args = ap.parse_args()
    from paper_2510_04286_b200 import synth
    lc = synth.CONFIGS[args.config]
    if args.impl == "reference":
        run_reference(args, lc)
    else:
        run_ours(args, lc)


if __name__ == "__main__":
    main()
