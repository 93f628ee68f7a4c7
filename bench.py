#!/usr/bin/env python
"""Throughput of the SliceMoE layer forward on B200, one JSON line per run.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg1] [--impl ours|reference] [--staged] [--backward]

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

# dram__bytes_read.sum + dram__bytes_write.sum per launch from ncu captures of the timed kernel, with the summary
# that holds them.  Not scaled between workloads: whether the expert pass's gathers and reductions hit L2 depends
# on the batch (cfg1's 16.8 MB of tokens stay in L2 and h' is still there when the kernel ends; cfg2's 134 MB do
# not).  A workload without a capture of its own reports traffic = null.
NCU_TRAFFIC = {
    # (kernel, N, ds, k, F): (bytes per launch, summary)
    ("forward_one_launch", 16384 * 8, 64, 2, 256): (17.9745e6 + 0.04e6, "profiles/pp_forward_kernel_cfg1_cfg2.md (ncu, cfg1)"),
    ("forward_one_launch", 65536 * 16, 64, 2, 256): (613.103e6 + 342.652e6, "profiles/pp_forward_kernel_cfg1_cfg2.md (ncu, cfg2)"),
    ("forward_one_launch", 128 * 32, 128, 2, 512): (17.868e6, "profiles/decode_forward_kernel_cfg4.md (ncu, cfg4)"),
    ("route", 32768 * 8, 256, 1, 1024): (134.453e6 + 87.19e6, "profiles/route_wide_kernel_cfg3.md (ncu, cfg3; 134.5 MB read + 87.2 MB of the zero rows of h', which the "
                                         "forward's router writes for the combine step and the stage's compulsory bytes do not count)"),
}
OTHER_CONFIGS = ("cfg2", "cfg3", "cfg3b", "cfg4", "paper768")     # paper768: the paper's own model shape (d = 768, S = 8, E = 16, k = 2)
# dram__bytes_read + dram__bytes_write of the two backward kernels on cfg1 (profiles/backward_cfg1.md)
NCU_TRAFFIC_BACKWARD_CFG1 = (43.363072e6 + 26.524160e6) + (87.232256e6 + 5.461248e6)
NCU_TRAFFIC_ROWS_CFG1 = 16384 * 8


def ncu_traffic(kernel, lc):
    """(DRAM bytes per launch of this workload's own capture, where the figure comes from) or (None, None)."""
    ent = NCU_TRAFFIC.get((kernel, lc.N, lc.ds, lc.k, lc.F))
    return ent if ent is not None else (None, None)


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
def layer_work(lc, kept_rows, touched_experts, w=None):
    """`w`: the weight tensors the forward is given; a bias passed as NULL is not counted as compulsory traffic."""
    b = 2 if lc.dtype == "bf16" else 4
    ds = lc.ds
    has = (lambda n: w.get(n) is not None) if w is not None else (lambda n: True)
    router_flops = 2.0 * lc.N * (ds * lc.Hr + lc.Hr * lc.E)
    expert_flops = 4.0 * kept_rows * ds * lc.F
    io_bytes = 2.0 * lc.T * lc.d * b
    router_w = (lc.Hr * ds + lc.Hr * has("br1") + lc.E * lc.Hr + lc.E * has("br2")) * b
    expert_w = touched_experts * (2 * ds * lc.F + lc.F * has("b1") + ds * has("b2")) * b
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
    """Streams SM clocks and throttle reasons from one `nvidia-smi -lms 100` child (read-only queries) while
    the bench runs; every sample is stamped on arrival so that a summary can cover one timed region only."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    NAMES = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")

    def __init__(self, gpu_id):
        self.gpu = gpu_id
        self.samples = []           # (arrival time, [fields])
        self.proc = None
        self._thread = None

    def _run(self):
        for line in self.proc.stdout:
            f = [x.strip() for x in line.strip().split(",")]
            if len(f) >= 6:
                self.samples.append((time.perf_counter(), f))

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return self
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()
        return self

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()           # the one child started above
            try:
                self.proc.wait(timeout=10)
            except Exception:
                self.proc.kill()
            self._thread.join(timeout=10)
            self.proc = None

    def summary(self, t0=None, t1=None):
        """Median SM clock and the throttle reasons seen between t0 and t1 (time.perf_counter values);
        without bounds, over every sample."""
        mhz, mx, reasons = [], None, set()
        for t, s in list(self.samples):
            if (t0 is not None and t < t0) or (t1 is not None and t > t1):
                continue
            try:
                mhz.append(float(s[0]))
                mx = float(s[1])
                for name, v in zip(self.NAMES, s[2:6]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                continue
        if mx is None and self.samples:
            try:
                mx = float(self.samples[-1][1][1])
            except Exception:
                pass
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
        "config": workload_config(lc),
        "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")},
        "e2e": {"value": r["value"], "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(lc):
    """The same dict in both arms (the GPU arm's cache policy is a fixed key, its details are in `buffer_rotation`)."""
    return {"workload": lc.name, "T": lc.T, "d": lc.d, "S": lc.S, "E": lc.E, "k": lc.k, "F": lc.F,
            "Hr": lc.Hr, "act": "gelu_tanh" if lc.act else "relu", "capacity": lc.capacity,
            "l2_gpu_arm": "distinct buffer sets larger than L2 rotate between steps"}


def l2_note(sets, wsets):
    note = (f"rotating {sets} distinct token/output buffer sets between steps (larger than the 126 MB L2)"
            if sets > 1 else "single buffer set (the weights one step reads exceed the L2)")
    if wsets > 1:
        note += f" and {wsets} copies of the weights (token sets alone would fit in L2 beside them)"
    return note


# --------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------
class Workload:
    """Device tensors of one workload (rotating token/output sets, weight copies, workspace) and the timed
    legs over them.  Every rank draws its own batches: rank r, set s uses seed 1000 r + s."""

    def __init__(self, sm, lc, rank):
        import torch
        from paper_2510_04286_b200 import synth, tensors
        self.sm, self.lc, self.torch = sm, lc, torch
        self.cfg = cfg = tensors.config_from_synth(lc)
        tdt = sm.torch_dtype(cfg)
        b = 2 if lc.dtype == "bf16" else 4
        set_bytes = 2 * lc.T * lc.d * b
        expert_w_bytes = 2.0 * lc.E * lc.F * lc.ds * b
        self.per_expert_streams = expert_w_bytes > 4e9
        if self.per_expert_streams:
            # weights far larger than L2 (and than one host draw): one token set; the experts the router
            # picks are drawn one at a time from their own seeded streams, the others are never read
            self.sets = self.wsets = 1
            wr = synth.make_router_weights(lc)
            w = tensors.weights_to_torch(wr, lc.dtype, drop_zero_biases=True)
            w["W1"] = torch.zeros((lc.E, lc.F, lc.ds), dtype=tdt, device="cuda")
            w["W2"] = torch.zeros((lc.E, lc.ds, lc.F), dtype=tdt, device="cuda")
            w["b1"] = w["b2"] = None
            self.w_all = [w]
        else:
            self.sets = int(max(2, min(64, -(-2.2 * L2_BYTES // set_bytes)))) if set_bytes < 2.2 * L2_BYTES else 2
            # (the named bf16 workloads have no biases: their all-zero bias tensors are passed as NULL, the
            # interface's "no bias"; a workload with real biases keeps them)
            w = tensors.weights_to_torch(synth.make_weights(lc), lc.dtype, drop_zero_biases=True)
            # Small batches (decode) would leave everything L2-resident however many token sets rotate: the
            # weights, their largest input, rotate too until tokens + weights exceed 2.2 x L2.
            w_bytes = sum(int(t.numel()) * t.element_size() for t in w.values() if t is not None)
            short = 2.2 * L2_BYTES - self.sets * set_bytes
            self.wsets = int(max(1, min(16, -(-short // w_bytes)))) if short > 0 else 1
            self.w_all = [w] + [{n: (None if t is None else t.clone()) for n, t in w.items()}
                                for _ in range(self.wsets - 1)]
        self.w = self.w_all[0]
        self.seeds = [1000 * rank + s for s in range(self.sets)]
        self.hs = [tensors.to_torch(synth.make_tokens(lc, seed=sd), lc.dtype) for sd in self.seeds]
        self.outs = [torch.empty((lc.T, lc.d), dtype=tdt, device="cuda") for _ in range(self.sets)]
        self.ws = sm.alloc_workspace(cfg)
        self.assigned = torch.empty((lc.E,), dtype=torch.int32, device="cuda")
        self.kept = torch.empty((lc.E,), dtype=torch.int32, device="cuda")
        if self.per_expert_streams:
            idx = torch.empty((cfg.N, cfg.k), dtype=torch.int32, device="cuda")
            p = torch.empty((cfg.N, cfg.k), dtype=torch.float32, device="cuda")
            sm.slicemoe_route(cfg, self.w, self.hs[0], idx, p, self.assigned, ws=self.ws)
            for e in sorted(set(int(x) for x in idx.cpu().numpy().ravel())):
                we = synth.make_expert_weights(lc, e)
                self.w["W1"][e].copy_(tensors.to_torch(we["W1"], lc.dtype))
                self.w["W2"][e].copy_(tensors.to_torch(we["W2"], lc.dtype))
                del we

    def step(self, i):
        self.sm.slicemoe_forward(self.cfg, self.w_all[i % self.wsets], self.hs[i % self.sets],
                                 self.outs[i % self.sets], self.ws, self.assigned, self.kept)

    def warm_up(self, n):
        for i in range(n):
            self.step(i)
        self.torch.cuda.synchronize()
        st = self.sm.slicemoe_last_status(self.ws)
        if st != 0:
            raise RuntimeError(f"device status {st} after warm-up of {self.lc.name}")
        self.kept_rows = int(self.kept.sum().item())
        self.touched = int((self.kept > 0).sum().item())

    def timed(self, fn, steps, min_replays, min_seconds, barrier, graph=True):
        """Times `steps` calls of fn(i) as one unit, replayed at least min_replays times and for at least
        min_seconds of device time, one CUDA-event pair per replay.  The unit is one CUDA graph of the
        steps (captured once) where capture works, else the plain launches.  Returns the per-replay seconds."""
        torch = self.torch
        replay, used_graph = None, False
        if graph:
            try:
                g = torch.cuda.CUDAGraph()
                # thread-local capture mode: CUDA calls of other threads (a process group's watchdog) do
                # not invalidate the capture
                with torch.cuda.graph(g, capture_error_mode="thread_local"):
                    for i in range(steps):
                        fn(i)
                replay, used_graph = g.replay, True
            except Exception as ex:          # say why and fall back to plain launches
                sys.stderr.write(f"graph capture failed, timing plain launches: {ex}\n")
        if replay is None:
            def replay():
                for i in range(steps):
                    fn(i)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        replay()
        barrier()
        e0.record(); replay(); e1.record()
        torch.cuda.synchronize()
        once = max(e0.elapsed_time(e1) / 1e3, 1e-6)
        n = int(max(min_replays, min(20000, -(-min_seconds // once))))
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        barrier()
        t0 = time.perf_counter()
        for a, b_ in ev:
            a.record(); replay(); b_.record()
        barrier()
        t1 = time.perf_counter()
        return [a.elapsed_time(b_) / 1e3 for a, b_ in ev], used_graph, (t0, t1)


def median(xs):
    xs = sorted(xs)
    return xs[len(xs) // 2]


def roofline_of(lc, work, peaks, t_step):
    """The layer's bound: the slower of its tensor time and its HBM time at the measured peaks."""
    t_tensor = work["total_flops"] / (peaks["bf16_tflops"] * 1e12)
    t_hbm = work["compulsory_bytes"] / (peaks["hbm_gbs"] * 1e9)
    bound = "tensor" if t_tensor >= t_hbm else "hbm"
    return dict(t_tensor=t_tensor, t_hbm=t_hbm, bound=bound, frac=max(t_tensor, t_hbm) / t_step)


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

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(local).uuid)
    except Exception:
        gpu_id = str(local)
    # one nvidia-smi child streams the clocks for the whole run; each summary below covers one timed region
    clocks = ClockSampler(gpu_id).start()
    b = 2 if lc.dtype == "bf16" else 4
    steps = max(1, args.steps)
    warm = max(10, args.warmup)
    wl = Workload(sm, lc, rank)
    cfg, w, hs, outs, ws, assigned, kept = wl.cfg, wl.w, wl.hs, wl.outs, wl.ws, wl.assigned, wl.kept
    sets, wsets = wl.sets, wl.wsets
    wl.warm_up(warm)
    kept_rows, touched = wl.kept_rows, wl.touched
    # routing balance of this batch (Eq. 2 with alpha = 0.1, Section 4's ELE), computed on the device
    stats = torch.empty(2, dtype=torch.float64, device="cuda")
    sm.slicemoe_load_stats(assigned, 0.1, stats)
    l_cap, ele = (float(x) for x in stats.cpu())

    # ---- timed region 1: device-resident inputs; the K steps as one CUDA graph, >= 100 replays ----------
    launches0 = sm.slicemoe_launch_count()
    for i in range(steps):
        wl.step(i)
    launches = sm.slicemoe_launch_count() - launches0           # launches of K steps (counted outside capture)
    t_replays, use_graph, window = wl.timed(wl.step, steps, args.replays, args.min_seconds, barrier)
    clk = clocks.summary(*window)

    # the same K steps as plain launches, once (the gaps between launches are the host's)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    start.record()
    for i in range(steps):
        wl.step(i)
    stop.record()
    barrier()
    t_plain = start.elapsed_time(stop) / 1e3

    # the same steps on ONE buffer set (tokens, outputs and weights stay in L2 where they fit): reported
    # beside the rotating (cold) figure, never as `value`
    t_warm, _, _ = wl.timed(lambda i: sm.slicemoe_forward(cfg, w, hs[0], outs[0], ws, assigned, kept),
                            steps, 10, 0.0, barrier)

    # ---- timed region 2: host buffers through the C ABI (K calls per repeat, 5 repeats) ---------------
    h_host = [tensors.to_torch(synth.make_tokens(lc, seed=wl.seeds[s]), lc.dtype, "cpu", pin=True)
              for s in range(min(sets, 4))]
    o_host = [torch.empty_like(x).pin_memory() for x in h_host]
    t_e2e, _, _ = wl.timed(lambda i: sm.slicemoe_forward_host(cfg, w, h_host[i % len(h_host)], o_host[i % len(h_host)],
                                                              ws, assigned, kept),
                           steps, 5, 0.0, barrier, graph=False)

    # ---- timed region 3: per-stage CUDA events (recorded by the library on its stream) ----
    # (the stage-timed call keeps one launch per stage; the forward timed above is one launch where the
    # shape has a single-kernel path)
    ev = [sm.StageEvents() for _ in range(min(steps, 64))]
    for i in range(3):
        sm.slicemoe_forward_profiled(cfg, w, hs[i % sets], outs[i % sets], ws, ev[0], assigned, kept)
    barrier()
    for i in range(len(ev)):
        sm.slicemoe_forward_profiled(cfg, wl.w_all[i % wsets], hs[i % sets], outs[i % sets], ws, ev[i], assigned, kept)
    torch.cuda.synchronize()
    stage_ms = np.median([e.stage_ms() for e in ev], axis=0)

    # ---- --staged: the four staged calls of the C ABI one by one (route, dispatch, expert_ffn, combine) -----
    # Not part of `value` (the forward call above is one launch): each call's median time over the rotating
    # batches and its algorithmic bytes / FLOPs, i.e. the achieved HBM GB/s of dispatch and combine.
    staged = None
    if args.staged:
        nb = min(sets, 4)
        st_idx = [torch.empty((cfg.N, cfg.k), dtype=torch.int32, device="cuda") for _ in range(nb)]
        st_p = [torch.empty((cfg.N, cfg.k), dtype=torch.float32, device="cuda") for _ in range(nb)]
        st_kept = torch.empty((cfg.E,), dtype=torch.int32, device="cuda")
        st_off = torch.empty((cfg.E + 1,), dtype=torch.int32, device="cuda")
        st_dest = [torch.empty((cfg.N, cfg.k), dtype=torch.int32, device="cuda") for _ in range(nb)]
        st_perm = torch.empty((max(cfg.R, 1),), dtype=torch.int32, device="cuda")
        st_x = [torch.empty((max(cfg.R, 1), cfg.ds), dtype=sm.torch_dtype(cfg), device="cuda") for _ in range(nb)]
        st_y = [torch.empty((max(cfg.R, 1), cfg.ds), dtype=sm.torch_dtype(cfg), device="cuda") for _ in range(nb)]
        calls = {
            "route": lambda i: sm.slicemoe_route(cfg, w, hs[i % nb], st_idx[i % nb], st_p[i % nb], assigned, None, ws),
            "dispatch": lambda i: sm.slicemoe_dispatch(cfg, hs[i % nb], st_idx[i % nb], st_p[i % nb], st_kept, st_off,
                                                       st_dest[i % nb], st_perm, st_x[i % nb], ws),
            "expert_ffn": lambda i: sm.slicemoe_expert_ffn(cfg, w, st_x[i % nb], st_off, st_y[i % nb], ws),
            "combine": lambda i: sm.slicemoe_combine(cfg, st_y[i % nb], st_dest[i % nb], outs[i % nb]),
        }
        for i in range(nb):                      # every buffer set holds a consistent chain before anything is timed
            for fn in calls.values():
                fn(i)
        torch.cuda.synchronize()
        staged = {}
        for name, fn in calls.items():
            ts, _, _ = wl.timed(fn, min(steps, 16), 10, 0.0, barrier)
            (t_call,) = max_over_ranks([median(ts) / min(steps, 16)], dist, device="cuda")
            staged[name] = t_call

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
        gouts = [tensors.to_torch(synth.make_grad_out(lc, seed=wl.seeds[s]), lc.dtype) for s in range(sets)]
        for s_ in range(sets):
            sm.slicemoe_forward(cfg, w, hs[s_], outs[s_], ws, assigned, kept, idxs[s_], gates[s_])
        shapes = dict(dWr1=(cfg.Hr, cfg.ds), dbr1=(cfg.Hr,), dWr2=(cfg.E, cfg.Hr), dbr2=(cfg.E,),
                      dW1=(cfg.E, cfg.F, cfg.ds), db1=(cfg.E, cfg.F), dW2=(cfg.E, cfg.ds, cfg.F), db2=(cfg.E, cfg.ds))
        grads = {n: torch.empty(sh, dtype=torch.float32, device="cuda") for n, sh in shapes.items()}
        bsteps = max(1, min(steps, 10))

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

    # every figure is the slowest rank's
    t_med, t_min, t_plain, t_same, t_e2e_med = max_over_ranks(
        [median(t_replays), min(t_replays), t_plain, median(t_warm), median(t_e2e)], dist, device="cuda")

    peaks, peak_src = load_peaks()
    others = {}
    if world == 1 and not args.no_other_configs:
        # the other single-GPU workloads, a few steps each (same protocol, fewer replays)
        w = {n: (None if t is None else True) for n, t in w.items()}      # (which tensors were passed: used below)
        del wl, hs, outs, ws
        for name in OTHER_CONFIGS:
            if name == lc.name:
                continue
            torch.cuda.empty_cache()
            olc = synth.CONFIGS[name]
            try:
                o = Workload(sm, olc, rank)
                o.warm_up(10)
                l0 = sm.slicemoe_launch_count()
                o.step(0)
                per_step = sm.slicemoe_launch_count() - l0
                ts, g, _ = o.timed(o.step, 10, 20, 0.05, barrier)
                ow = layer_work(olc, o.kept_rows, o.touched, o.w)
                rf = roofline_of(olc, ow, peaks, median(ts) / 10)
                others[name] = {"ms_per_step": 1e3 * median(ts) / 10, "ms_per_step_min": 1e3 * min(ts) / 10,
                                "steps": 10, "replays": len(ts), "bound": rf["bound"], "frac": rf["frac"],
                                "t_tensor_us": 1e6 * rf["t_tensor"], "t_hbm_us": 1e6 * rf["t_hbm"],
                                "tokens_per_s": olc.T * 10 / median(ts), "gpu_launches_per_step": int(per_step),
                                "buffer_rotation": l2_note(o.sets, o.wsets),
                                "timing": "CUDA graph" if g else "plain launches"}
                del o
            except Exception as ex:
                others[name] = {"error": str(ex)[:200]}
    clocks.stop()

    if rank == 0:
        work = layer_work(lc, kept_rows, touched, w)
        stages = dict(zip(sm.STAGES, (float(x) for x in stage_ms)))
        t_step = t_med / steps
        single_launch = launches == steps
        layer = roofline_of(lc, work, peaks, t_step)
        if single_launch:
            # the timed forward is ONE kernel (router, dispatch and expert phases): its launch duration is
            # the step time the events measure, and its bound is the layer's (tensor or HBM, whichever is slower)
            dom = "forward_one_launch"
            kernel_ms = 1e3 * t_step
            if layer["bound"] == "tensor":
                roof = {"bound": "tensor", "achieved": work["total_flops"] / t_step / 1e12,
                        "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"}
            else:
                roof = {"bound": "hbm", "achieved": work["compulsory_bytes"] / t_step / 1e9,
                        "peak": peaks["hbm_gbs"], "unit": "GB/s"}
            compulsory = work["compulsory_bytes"]
        else:
            dom = max(stages, key=stages.get)
            kernel_ms = stages[dom]
            fl = work["stage_flops"].get(dom, 0.0) / (peaks["bf16_tflops"] * 1e12)
            by = work["stage_bytes"][dom] / (peaks["hbm_gbs"] * 1e9)
            if fl >= by:
                roof = {"bound": "tensor", "achieved": work["stage_flops"][dom] / (kernel_ms * 1e-3) / 1e12,
                        "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"}
            else:
                roof = {"bound": "hbm", "achieved": work["stage_bytes"][dom] / (kernel_ms * 1e-3) / 1e9,
                        "peak": peaks["hbm_gbs"], "unit": "GB/s"}
            compulsory = work["stage_bytes"][dom]
        traffic, traffic_src = ncu_traffic(dom, lc)
        roof.update(frac=roof["achieved"] / roof["peak"], traffic=traffic, traffic_source=traffic_src,
                    traffic_over_compulsory=(traffic / compulsory if traffic else None),
                    compulsory_bytes=compulsory, kernel=dom, kernel_ms=kernel_ms, peak_source=f"of {peak_src}")
        mhz = clk["sm_mhz"]
        line = {
            "metric": "SliceMoE layer fwd tokens/s", "value": aggregate(shard_tokens(lc.T, world), steps, [t_med]),
            "unit": "tokens/s", "n_gpus": world, "steps": steps, "warmup": warm,
            "ms_per_step": 1e3 * t_step, "ms_per_step_min": 1e3 * t_min / steps, "replays": len(t_replays),
            "timing": (("one CUDA graph of the K steps" if use_graph else "K plain launches (graph capture failed)")
                       + ", one event pair per replay; value and ms_per_step are the median replay"),
            "timed_seconds": sum(t_replays),
            "sm_cycles_per_step": (t_step * mhz * 1e6 if mhz else None),
            "ms_per_step_plain_launches": 1e3 * t_plain / steps,
            "ms_per_step_same_buffers": 1e3 * t_same / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": lc.dtype, "data": "synthetic", "config": workload_config(lc),
            "buffer_rotation": l2_note(sets, wsets),
            "routed_slices_per_s": world * lc.R / t_step,
            "routing_stats": {"ele": ele, "l_cap_alpha_0.1": l_cap},
            "e2e": {"value": world * lc.T * steps / t_e2e_med, "unit": "tokens/s",
                    "h2d_bytes_per_step": lc.T * lc.d * b, "d2h_bytes_per_step": lc.T * lc.d * b},
            "gpu_launches": int(launches),
            "clocks": clk,
            "roofline": roof,
            "stage_ms_one_launch_per_stage": stages,
            "activation_bound": {
                "what": "tanh unit: R_kept*F GELU(tanh) evaluations at 16 per clock per SM",
                "t_us": (1e6 * kept_rows * lc.F / (N_SM * TANH_PER_CLK_PER_SM) / (clk["sm_max_mhz"] or 1965.0) / 1e6
                         if lc.act else 0.0)},
            "layer_roofline": {"t_tensor_us": 1e6 * layer["t_tensor"], "t_hbm_us": 1e6 * layer["t_hbm"],
                               "bound": layer["bound"], "frac": layer["frac"], "kept_rows": kept_rows,
                               "touched_experts": touched, "peak_source": f"of {peak_src}"},
        }
        if staged is not None:
            sb, sf = work["stage_bytes"], work["stage_flops"]
            line["staged_calls"] = {
                name: {"ms": 1e3 * t, "hbm_gbs": sb[name] / t / 1e9, "frac_of_hbm": sb[name] / t / 1e9 / peaks["hbm_gbs"],
                       **({"tflops": sf[name] / t / 1e12} if name in sf else {})}
                for name, t in staged.items()}
        if others:
            line["other_configs"] = others
        if bwd is not None:
            # algorithmic work of a backward = twice the forward's (input and weight gradient of every
            # product); the kernels also redo the forward's products (recompute factor 1.5).  fp32 on
            # CUDA cores: the bound is the FMA pipes, 128 lanes x 2 FLOP per clock per SM.
            alu_peak = N_SM * 128 * 2 * (clk["sm_max_mhz"] or 1965.0) * 1e6 / 1e12
            ach = 2.0 * work["total_flops"] / bwd["t"] / 1e12
            line["backward"] = {
                "ms_per_step": 1e3 * bwd["t"], "tokens_per_s": world * lc.T / bwd["t"], "steps": bwd["steps"],
                "gpu_launches_per_step": int(bwd["launches_per_step"]), "dtype": "f32",
                "roofline": {"bound": "alu", "achieved": ach, "peak": alu_peak, "unit": "TFLOP/s",
                             "frac": ach / alu_peak,
                             "traffic": (NCU_TRAFFIC_BACKWARD_CFG1 * lc.N / NCU_TRAFFIC_ROWS_CFG1
                                         if lc.ds == 64 and lc.k == 2 and lc.F == 256 else None),
                             "traffic_source": "profiles/backward_cfg1.md (ncu, cfg1, scaled by rows)",
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
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the short runs of the other single-GPU workloads (the `other_configs` object)")
    ap.add_argument("--replays", type=int, default=100, help="least number of timed replays of the K steps")
    ap.add_argument("--min-seconds", type=float, default=2.0,
                    help="least device time of the timed region (more replays are added to reach it)")
    ap.add_argument("--staged", action="store_true",
                    help="also time the four staged calls one by one (the `staged_calls` object: ms and achieved HBM GB/s)")
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
