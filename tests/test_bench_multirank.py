"""The N > 1 host logic of bench.py on CPU: two gloo ranks, replicas only (no data-path collective)."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    import torch.distributed as dist
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r "measures" (r + 1) seconds on the device-resident arm and (r + 2) on the host arm
    t_dev, t_e2e = bench.max_over_ranks([rank + 1.0, rank + 2.0], dist)
    dist.barrier()
    if rank == 0:
        tokens = bench.shard_tokens(1000, world)
        out.put((t_dev, t_e2e, tokens, bench.aggregate(tokens, 10, [t_dev])))
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_sum_the_tokens():
    torch = pytest.importorskip("torch")
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    t_dev, t_e2e, tokens, value = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert (t_dev, t_e2e) == (2.0, 3.0)              # max over ranks
    assert tokens == [1000, 1000]                    # weak scaling: every rank its own batch
    assert value == 2 * 1000 * 10 / 2.0              # whole-job tokens / slowest rank


def test_single_rank_helpers():
    import bench
    assert bench.max_over_ranks([0.5, 0.25]) == [0.5, 0.25]
    assert bench.aggregate([100], 4, [2.0]) == 200.0
    from paper_2510_04286_b200 import synth
    w = bench.layer_work(synth.CONFIGS["cfg1"], kept_rows=262144, touched_experts=16)
    assert abs(w["total_flops"] - 22.55e9) < 0.01e9          # router 5.37 G + experts 17.18 G
    assert abs(w["compulsory_bytes"] - 34.7e6) < 0.1e6
    # a workload reports the DRAM traffic of its own ncu capture only (nothing is scaled from another batch size);
    # absent biases are not compulsory bytes
    cfg1, cfg2 = synth.CONFIGS["cfg1"], synth.CONFIGS["cfg2"]
    key = ("probe", cfg1.N, cfg1.ds, cfg1.k, cfg1.F)
    bench.NCU_TRAFFIC[key] = (100e6, "a summary")
    try:
        assert bench.ncu_traffic("probe", cfg1) == (100e6, "a summary")
        assert bench.ncu_traffic("probe", cfg2) == (None, None)
        assert bench.ncu_traffic("no such kernel", cfg1) == (None, None)
    finally:
        del bench.NCU_TRAFFIC[key]
    no_bias = {"Wr1": 1, "Wr2": 1, "W1": 1, "W2": 1, "br1": None, "br2": None, "b1": None, "b2": None}
    w0 = bench.layer_work(cfg1, kept_rows=262144, touched_experts=16, w=no_bias)
    assert w["compulsory_bytes"] - w0["compulsory_bytes"] == 2 * (256 + 16 + 16 * (256 + 64))
    r = bench.roofline_of(synth.CONFIGS["cfg1"], w, {"bf16_tflops": 1000.0, "hbm_gbs": 1000.0}, 1e-4)
    assert r["bound"] == "hbm" and r["frac"] == pytest.approx(w["compulsory_bytes"] / 1e12 / 1e-4)
    s = bench.ClockSampler("0")
    s.samples = [(1.0, ["1900", "1965", "Not Active", "Not Active", "Not Active", "Active"]),
                 (2.0, ["1800", "1965", "Not Active", "Not Active", "Not Active", "Not Active"]),
                 (3.0, ["1700", "1965", "Active", "Not Active", "Not Active", "Not Active"])]
    assert s.summary(0.5, 2.5) == {"sm_mhz": 1900.0, "sm_max_mhz": 1965.0, "reasons": ["sw_power_cap"], "samples": 2}
    assert s.summary()["reasons"] == ["hw_slowdown", "sw_power_cap"]
    assert bench.median([3.0, 1.0, 2.0]) == 2.0
