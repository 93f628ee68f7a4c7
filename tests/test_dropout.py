"""Section 3.3, cross-slice dropout: pins of the oracle (CPU) and GPU parity."""
import numpy as np
import pytest

import oracle
from paper_2510_04286_b200 import synth

# Known-answer vectors of Philox4x32-10 from the Random123 distribution (Salmon, Moraes, Dror, Shaw,
# "Parallel random numbers: as easy as 1, 2, 3", SC'11): counter, key -> output.
PHILOX_KAT = [
    ((0, 0, 0, 0), (0, 0), (0x6627E8D5, 0xE169C58D, 0xBC57AC4C, 0x9B00DBD8)),
    ((0xFFFFFFFF,) * 4, (0xFFFFFFFF,) * 2, (0x408F276D, 0x41C83B0E, 0xA20BC7C6, 0x6D5451FD)),
    ((0x243F6A88, 0x85A308D3, 0x13198A2E, 0x03707344), (0xA4093822, 0x299F31D0),
     (0xD16CFE09, 0x94FDCCEB, 0x5001E420, 0x24126EA1)),
]


def some_topk_p(N, k, seed=0):
    rng = np.random.default_rng(seed)
    p = rng.dirichlet(np.ones(k + 3), size=N)[:, :k]
    return -np.sort(-p, axis=1)                      # descending, sums below 1 like real top-k


@pytest.mark.parametrize("ctr,key,want", PHILOX_KAT)
def test_philox_known_answers(ctr, key, want):
    assert tuple(int(x) for x in oracle.philox4x32(ctr, key)) == want


def test_dropout_brute_force_from_the_generator():
    """Pure-Python restatement on a small input: draw, compare, renormalise."""
    N, k, seed, rate = 40, 3, 0x1234_5678_9ABC, 0.2
    p = some_topk_p(N, k)
    got, dropped = oracle.gate_dropout(p, seed, rate)
    thr = int(rate * 2 ** 32)
    for n in range(N):
        words = [int(oracle.philox4x32((n, j, 0, 0), (seed & 0xFFFFFFFF, seed >> 32))[0]) for j in range(k)]
        drop = [w < thr for w in words]
        assert drop == list(dropped[n])
        kept = [p[n, j] for j in range(k) if not drop[j]]
        want = [1.0] + [0.0] * (k - 1) if not kept else [0.0 if drop[j] else p[n, j] / sum(kept) for j in range(k)]
        assert got[n] == pytest.approx(want, rel=1e-15, abs=0)


def test_dropout_invariants():
    p = some_topk_p(50000, 2)
    out, dropped = oracle.gate_dropout(p, 7, 0.2)
    assert np.allclose(out.sum(1), 1.0, atol=1e-15)                  # survivors renormalised, or top-1 = 1
    assert np.all(out[dropped & ~dropped.all(1, keepdims=True)] == 0.0)
    all_dropped = dropped.all(1)
    assert np.all(out[all_dropped, 0] == 1.0) and np.all(out[all_dropped, 1:] == 0.0)
    # survivors keep their ratio
    both = ~dropped.any(1)
    assert np.allclose(out[both, 0] / out[both, 1], p[both, 0] / p[both, 1], rtol=1e-12)
    # the drop frequency is the rate (binomial, 5 sigma), and the two assignments draw independently
    n = dropped.size
    assert abs(dropped.mean() - 0.2) < 5 * np.sqrt(0.2 * 0.8 / n)
    assert abs(all_dropped.mean() - 0.04) < 5 * np.sqrt(0.04 * 0.96 / len(p))


def test_dropout_limits_and_determinism():
    p = some_topk_p(1000, 3)
    out0, d0 = oracle.gate_dropout(p, 1, 0.0)
    assert not d0.any() and np.allclose(out0, p / p.sum(1, keepdims=True), rtol=1e-15)   # rate 0: renormalise only
    out1, d1 = oracle.gate_dropout(p, 1, 1.0)
    assert d1.all() and np.all(out1[:, 0] == 1.0) and not out1[:, 1:].any()             # all dropped: top-1 = 1
    a, da = oracle.gate_dropout(p, 99, 0.3)
    b, db = oracle.gate_dropout(p, 99, 0.3)
    c, dc = oracle.gate_dropout(p, 100, 0.3)
    assert np.array_equal(da, db) and np.array_equal(a, b) and not np.array_equal(da, dc)
    # the draw of (n, j) depends on (seed, n, j) only: a prefix of the rows gives the same mask
    _, dprefix = oracle.gate_dropout(p[:100], 99, 0.3)
    assert np.array_equal(dprefix, da[:100])


@pytest.mark.gpu
@pytest.mark.parametrize("k,rate,seed", [(1, 0.2, 3), (2, 0.2, 2 ** 40 + 17), (3, 0.5, 11), (2, 0.0, 5), (2, 1.0, 5), (8, 0.2, 1)])
def test_gpu_gate_dropout_matches_oracle(k, rate, seed):
    import torch
    from paper_2510_04286_b200 import binding, tensors
    N = 70001
    lc = synth.LayerConfig("drop", T=N, d=64, S=1, E=16, k=k, F=256)
    cfg = tensors.config_from_synth(lc)
    p = some_topk_p(N, k, seed=k).astype(np.float32)
    want, dropped = oracle.gate_dropout(p.astype(np.float64), seed, rate)
    t = torch.from_numpy(p.copy()).cuda()
    binding.slicemoe_gate_dropout(cfg, t, seed, rate)
    torch.cuda.synchronize()
    got = t.cpu().numpy()
    assert np.array_equal(got == 0.0, want == 0.0)                   # the same assignments dropped, bit for bit
    assert np.abs(got - want).max() <= 2e-7                          # one fp32 division against fp64


@pytest.mark.gpu
def test_gpu_train_mode_staged_forward():
    """route -> gate_dropout -> dispatch -> expert_ffn -> combine on the GPU against the same chain of
    oracle calls (dropped assignments stay routed with gate 0)."""
    import torch
    from paper_2510_04286_b200 import binding, tensors
    import parity_util as pu
    lc = synth.CONFIGS["cfg1"].with_tokens(300)
    h, w = synth.make_layer_inputs(lc, 0)
    gpu = pu.GpuLayer(lc, h, w)
    ocfg = pu.oracle_config(lc)
    ref_route = oracle.route(ocfg, h, w)
    idx = torch.from_numpy(ref_route["topk_idx"]).cuda()            # routing itself is graded elsewhere
    p = torch.from_numpy(ref_route["topk_p"].astype(np.float32)).cuda()
    binding.slicemoe_gate_dropout(gpu.cfg, p, 2024, 0.2)
    kept, offsets, dest, perm, xperm = gpu.dispatch(idx, p)
    h_out = gpu.combine(gpu.expert_ffn(xperm, offsets), dest)
    torch.cuda.synchronize()
    gates, _ = oracle.gate_dropout(ref_route["topk_p"].astype(np.float32).astype(np.float64), 2024, 0.2)
    d = oracle.dispatch(ocfg, ref_route["topk_idx"])
    n_kept = int(d["offsets"][-1])
    x = oracle.weight_slices(ocfg, h, gates, d["dest"], n_kept)
    y = oracle.expert_ffn(ocfg, x, d["offsets"], w)
    want = oracle.combine(ocfg, y, d["dest"])
    pu.assert_outputs_close(tensors.to_numpy_f32(h_out), want, lc.dtype, "train-mode h'")


@pytest.mark.gpu
@pytest.mark.parametrize("name,rate,seed", [
    ("cfg1", 0.2, 7),          # 64-wide slices: gates drawn inside the one-launch forward
    ("cfg1", 0.0, 3),          # rate 0 still re-normalises the k probabilities
    ("cfg1", 1.0, 5),          # everything dropped: the top-1 assignment gets weight 1
    ("cfg3b", 0.3, 11),        # capacity limit, ds = 256, k = 1: stage-by-stage form with the gate step
    ("cfg4", 0.2, 13),         # decode shape: stage-by-stage form
    ("cfg0", 0.5, 17),         # fp32 storage, ReLU, biases: CUDA-core kernels
])
def test_gpu_train_mode_forward(name, rate, seed):
    """slicemoe_forward with cfg.train_gates: the returned gates are Section 3.3's (masks equal to the oracle's
    draw for draw, survivors re-normalised) and h' is the layer evaluated with those gates."""
    import dataclasses
    import torch
    from paper_2510_04286_b200 import binding, tensors
    import parity_util as pu
    lc = synth.CONFIGS[name].with_tokens(300 if name != "cfg4" else 64)
    h, w = synth.make_layer_inputs(lc, 0)
    gpu = pu.GpuLayer(lc, h, w)
    plain = gpu.forward()
    gpu.cfg = dataclasses.replace(gpu.cfg, train_gates=1, dropout_rate=rate, dropout_seed=seed)
    h_out, assigned, kept, idx, gates = gpu.forward()
    torch.cuda.synchronize()
    assert gpu.status() == 0
    idx_np, g_np = idx.cpu().numpy(), gates.cpu().numpy().astype(np.float64)
    assert np.array_equal(idx_np, plain[3].cpu().numpy())                  # the draw does not touch the routing
    # gates: the oracle's rule applied to the probabilities the plain forward returned for the same picks
    p_plain = plain[4].cpu().numpy()
    want_g, dropped = oracle.gate_dropout(p_plain.astype(np.float64), seed, rate)
    none = dropped.all(axis=1)
    assert np.array_equal(g_np == 0.0, np.where(none[:, None], np.arange(lc.k)[None, :] > 0, dropped))
    assert np.abs(g_np - want_g).max() <= 4e-7                             # one fp32 division against fp64
    # h': the oracle's chain with the GPU's picks and gates
    ocfg = pu.oracle_config(lc)
    d = oracle.dispatch(ocfg, idx_np)
    assert np.array_equal(kept.cpu().numpy(), d["kept"])
    n_kept = int(d["offsets"][-1])
    x = oracle.weight_slices(ocfg, h, g_np, d["dest"], n_kept)
    y = oracle.expert_ffn(ocfg, x, d["offsets"], w)
    want = oracle.combine(ocfg, y, d["dest"])
    pu.assert_outputs_close(tensors.to_numpy_f32(h_out), want, lc.dtype, "train-mode h'", one_ulp_of_element=True)
    # a refused rate
    bad = dataclasses.replace(gpu.cfg, dropout_rate=1.5)
    gpu.cfg = bad
    with pytest.raises(binding.SliceMoEError):
        gpu.forward()
