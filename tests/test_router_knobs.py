"""Router ablation knobs (softmax temperature, Figure 7; Gaussian logit noise, Figure 6) and shuffled
slices (Figure 5): the oracle against closed forms and invariants on the CPU, the CUDA path against
the oracle on the GPU."""
from dataclasses import replace

import numpy as np
import pytest

import oracle
from paper_2510_04286_b200 import synth

import parity_util as pu

LC = synth.LayerConfig
TINY = LC("knobs", T=24, d=64, S=4, E=8, k=2, F=32, Hr=16, dtype="f32", act=0, init="kaiming")


def _route(lc, h, w):
    return oracle.route(pu.oracle_config(lc), h, w)


def _log_odds(probs):
    lp = np.log(probs)
    return lp - lp[:, :1]


# ---------------------------------------------------------------- temperature (CPU) --------

def test_temperature_one_is_the_default():
    h, w = synth.make_layer_inputs(TINY, 0)
    a = _route(TINY, h, w)
    b = _route(replace(TINY, temperature=1.0), h, w)
    np.testing.assert_array_equal(a["probs"], b["probs"])
    np.testing.assert_array_equal(a["topk_idx"], b["topk_idx"])


@pytest.mark.parametrize("tau", [0.5, 2.0, 7.0])
def test_temperature_divides_the_log_odds(tau):
    # softmax(g / tau): log(p_i / p_j) = (g_i - g_j) / tau, so the log-odds shrink by exactly tau
    h, w = synth.make_layer_inputs(TINY, 1)
    base = _route(TINY, h, w)
    hot = _route(replace(TINY, temperature=tau), h, w)
    np.testing.assert_allclose(_log_odds(hot["probs"]) * tau, _log_odds(base["probs"]), rtol=0, atol=1e-10)
    np.testing.assert_allclose(hot["probs"].sum(axis=1), 1.0, atol=1e-12)
    np.testing.assert_array_equal(hot["topk_idx"], base["topk_idx"])      # a monotone map keeps the order


def test_temperature_limits():
    h, w = synth.make_layer_inputs(TINY, 2)
    flat = _route(replace(TINY, temperature=1e12), h, w)["probs"]
    np.testing.assert_allclose(flat, 1.0 / TINY.E, atol=1e-9)
    sharp = _route(replace(TINY, temperature=1e-4), h, w)
    base = _route(TINY, h, w)
    clear = base["gap"] > 1e-6
    assert clear.any()
    top1 = sharp["probs"][np.arange(TINY.N), base["topk_idx"][:, 0]]
    # the winner takes everything when its logit leads by more than a few tau
    lead = np.sort(_log_odds(base["probs"]), axis=1)
    lead = lead[:, -1] - lead[:, -2]
    np.testing.assert_allclose(top1[lead > 1e-2], 1.0, atol=1e-12)


def test_bad_knobs_are_rejected():
    h, w = synth.make_layer_inputs(TINY, 0)
    with pytest.raises(Exception):
        _route(replace(TINY, temperature=-1.0), h, w)
    with pytest.raises(Exception):
        _route(replace(TINY, noise_sigma=-0.5), h, w)


# ---------------------------------------------------------------- logit noise (CPU) --------

def test_noise_is_standard_normal():
    from scipy import stats
    xs = np.array([oracle.logit_noise(2024, n, e) for n in range(2500) for e in range(16)])
    assert abs(xs.mean()) < 4.0 / np.sqrt(xs.size)
    assert abs(xs.var() - 1.0) < 4.0 * np.sqrt(2.0 / xs.size)
    assert stats.kstest(xs, "norm").pvalue > 1e-3
    assert abs(stats.skew(xs)) < 0.06 and abs(stats.kurtosis(xs)) < 0.12
    grid = xs.reshape(2500, 16)
    # neighbours along either axis are uncorrelated, and another seed gives another stream
    assert abs(np.corrcoef(grid[:, 0], grid[:, 1])[0, 1]) < 0.08
    assert abs(np.corrcoef(grid[:-1, 3], grid[1:, 3])[0, 1]) < 0.08
    other = np.array([oracle.logit_noise(2025, n, 0) for n in range(2500)])
    assert abs(np.corrcoef(grid[:, 0], other)[0, 1]) < 0.08


def test_noise_draw_follows_the_stated_recipe():
    # Box-Muller on the two leading words of the (separately pinned) Philox block, 24-bit uniforms
    for seed, n, e in ((0, 0, 0), (5, 17, 3), ((1 << 40) + 9, 123456, 63)):
        x = oracle.philox4x32([n, e, 1, 0], [seed & 0xFFFFFFFF, seed >> 32])
        u0 = ((int(x[0]) >> 8) + 0.5) / 2.0 ** 24
        u1 = ((int(x[1]) >> 8) + 0.5) / 2.0 ** 24
        want = np.sqrt(-2.0 * np.log(u0)) * np.cos(2.0 * np.pi * u1)
        assert abs(oracle.logit_noise(seed, n, e) - want) < 1e-12


def test_zero_sigma_is_the_plain_router():
    h, w = synth.make_layer_inputs(TINY, 3)
    a = _route(TINY, h, w)
    b = _route(replace(TINY, noise_sigma=0.0, noise_seed=99), h, w)
    np.testing.assert_array_equal(a["probs"], b["probs"])


@pytest.mark.parametrize("tau", [0.0, 2.0])
def test_noise_shifts_the_log_odds_before_the_temperature(tau):
    # softmax((g + sigma eps) / tau): log-odds move by sigma (eps_e - eps_0) / tau for row n, expert e
    sigma, seed = 0.7, 31
    t = tau if tau > 0 else 1.0
    h, w = synth.make_layer_inputs(TINY, 4)
    base = _route(replace(TINY, temperature=tau), h, w)
    noisy = _route(replace(TINY, temperature=tau, noise_sigma=sigma, noise_seed=seed), h, w)
    eps = np.array([[oracle.logit_noise(seed, n, e) for e in range(TINY.E)] for n in range(TINY.N)])
    want = _log_odds(base["probs"]) + sigma * (eps - eps[:, :1]) / t
    np.testing.assert_allclose(_log_odds(noisy["probs"]), want, rtol=0, atol=1e-9)
    # the picks are the arg-top-k of the noisy probabilities
    order = np.argsort(-noisy["probs"], axis=1, kind="stable")[:, :TINY.k]
    np.testing.assert_array_equal(noisy["topk_idx"], order)
    assert (noisy["topk_idx"] != base["topk_idx"]).any()                 # sigma = 0.7 does move some picks


def test_noise_reaches_the_forward_and_the_sampled_rows():
    lc = replace(TINY, noise_sigma=0.5, noise_seed=7, temperature=1.5)
    h, w = synth.make_layer_inputs(lc, 5)
    ocfg = pu.oracle_config(lc)
    r = oracle.route(ocfg, h, w)
    f = oracle.forward(ocfg, h, w)
    np.testing.assert_array_equal(f["topk_idx"], r["topk_idx"])
    np.testing.assert_array_equal(f["probs"], r["probs"])
    pick = np.array([0, 5, 17, lc.N - 1])
    rows = oracle.rows(ocfg, h, w, pick, f["topk_idx"][pick], np.ones((4, lc.k), bool))
    np.testing.assert_allclose(rows["y"], f["h_out"].reshape(lc.N, lc.ds)[pick], atol=1e-12)


# ---------------------------------------------------------------- shuffled slices (CPU) ----

def test_permute_columns_worked_example():
    x = np.array([[10.0, 11.0, 12.0, 13.0], [20.0, 21.0, 22.0, 23.0]])
    perm = [2, 0, 3, 1]
    np.testing.assert_array_equal(oracle.permute_columns(x, perm), [[12, 10, 13, 11], [22, 20, 23, 21]])
    np.testing.assert_array_equal(oracle.permute_columns(x, perm, inverse=True), [[11, 13, 10, 12], [21, 23, 20, 22]])
    back = oracle.permute_columns(oracle.permute_columns(x, perm), perm, inverse=True)
    np.testing.assert_array_equal(back, x)
    with pytest.raises(ValueError):
        oracle.permute_columns(x, [0, 0, 1, 2])


def test_identity_permutation_is_the_plain_layer():
    h, w = synth.make_layer_inputs(TINY, 6)
    ocfg = pu.oracle_config(TINY)
    a = oracle.forward(ocfg, h, w)["h_out"]
    b = oracle.forward_shuffled(ocfg, h, w, np.arange(TINY.d))["h_out"]
    np.testing.assert_array_equal(a, b)


def test_moving_whole_slices_changes_nothing():
    # router and experts are shared by all slices: a permutation that only reorders whole slices,
    # undone on the output, is the plain layer
    h, w = synth.make_layer_inputs(TINY, 7)
    ocfg = pu.oracle_config(TINY)
    order = np.array([2, 0, 3, 1])
    perm = (order[:, None] * TINY.ds + np.arange(TINY.ds)[None, :]).ravel()
    a = oracle.forward(ocfg, h, w)["h_out"]
    b = oracle.forward_shuffled(ocfg, h, w, perm)["h_out"]
    np.testing.assert_array_equal(a, b)


def test_shuffle_inside_slices_equals_permuted_weights():
    # the same shuffle sigma inside every slice is absorbed by the weights: with the input columns
    # of Wr1 and W1, and the output rows of W2 and b2, reordered by sigma, the shuffled layer returns
    # the plain layer's h' (an inverse applied the wrong way round, or to the wrong side, fails here)
    rng = np.random.default_rng(0)
    sig = rng.permutation(TINY.ds)
    perm = (np.arange(TINY.S)[:, None] * TINY.ds + sig[None, :]).ravel()
    h, w = synth.make_layer_inputs(TINY, 8)
    ocfg = pu.oracle_config(TINY)
    w2 = dict(w)
    w2["Wr1"] = w["Wr1"][:, sig]
    w2["W1"] = w["W1"][:, :, sig]
    w2["W2"] = w["W2"][:, sig, :]
    w2["b2"] = w["b2"][:, sig]
    a = oracle.forward(ocfg, h, w)["h_out"]
    b = oracle.forward_shuffled(ocfg, h, w2, perm)["h_out"]
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-12)
    # a shuffle that mixes slices is a different layer
    mixed = rng.permutation(TINY.d)
    c = oracle.forward_shuffled(ocfg, h, w, mixed)["h_out"]
    assert np.abs(c - a).max() > 1e-3


# ---------------------------------------------------------------- CUDA path ----------------

GPU_SHAPES = {
    "bf16_tensor_core": LC("kn_tc", T=333, d=512, S=8, E=16, k=2, F=256),
    "bf16_wide_rows": LC("kn_w", T=70, d=512, S=2, E=16, k=2, F=512, Hr=128),
    "bf16_cuda_core": LC("kn_cc", T=90, d=96, S=4, E=4, k=1, F=64, Hr=64),       # ds = 24
    "f32": replace(synth.CONFIGS["cfg0"], T=200),
}


@pytest.mark.gpu
@pytest.mark.parametrize("name", list(GPU_SHAPES))
@pytest.mark.parametrize("tau", [0.5, 2.0])
def test_gpu_temperature(name, tau):
    import torch
    lc = replace(GPU_SHAPES[name], temperature=tau)
    h, w = synth.make_layer_inputs(lc, 0)
    gpu = pu.GpuLayer(lc, h, w)
    idx, p, assigned, probs = gpu.route()
    torch.cuda.synchronize()
    ref = _route(lc, h, w)
    pu.check_routing(ref["probs"], ref["gap"], ref["topk_idx"], idx.cpu().numpy(), p.cpu().numpy().astype(np.float64))
    assert np.abs(probs.cpu().numpy() - ref["probs"]).max() <= 2e-4
    rep = pu.check_forward_against_oracle(lc)
    assert rep["excluded"] < lc.N


@pytest.mark.gpu
@pytest.mark.parametrize("name", list(GPU_SHAPES))
def test_gpu_logit_noise(name):
    import torch
    lc = replace(GPU_SHAPES[name], noise_sigma=0.5, noise_seed=(3 << 32) + 11, temperature=1.5)
    h, w = synth.make_layer_inputs(lc, 1)
    gpu = pu.GpuLayer(lc, h, w)
    idx, p, assigned, probs = gpu.route()
    torch.cuda.synchronize()
    ref = _route(lc, h, w)
    pu.check_routing(ref["probs"], ref["gap"], ref["topk_idx"], idx.cpu().numpy(), p.cpu().numpy().astype(np.float64))
    assert np.abs(probs.cpu().numpy() - ref["probs"]).max() <= 2e-4
    clean = _route(replace(lc, noise_sigma=0.0), h, w)
    assert (clean["topk_idx"] != ref["topk_idx"]).any()
    pu.check_forward_against_oracle(lc, seed=1)


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("T,d", [(77, 256), (1000, 768), (5, 8192), (0, 64), (300, 16384)])
def test_gpu_permute_columns(dtype, T, d):
    import torch
    from paper_2510_04286_b200 import binding, tensors
    lc = LC("perm", T=T, d=d, S=1, E=1, k=1, F=8, dtype=dtype)
    cfg = tensors.config_from_synth(lc)
    rng = np.random.default_rng(d + T)
    perm_np = rng.permutation(d).astype(np.int32)
    x_np = synth.make_tokens(lc, 3)
    x = tensors.to_torch(x_np, dtype)
    perm = torch.from_numpy(perm_np).cuda()
    fwd = torch.empty_like(x)
    back = torch.empty_like(x)
    before = binding.slicemoe_launch_count()
    binding.slicemoe_permute_columns(cfg, x, fwd, perm)
    binding.slicemoe_permute_columns(cfg, fwd, back, perm, inverse=True)
    torch.cuda.synchronize()
    assert binding.slicemoe_launch_count() - before == (2 if T else 0)
    if T == 0:
        return
    np.testing.assert_array_equal(tensors.to_numpy_f32(fwd), oracle.permute_columns(x_np, perm_np))
    np.testing.assert_array_equal(tensors.to_numpy_f32(back), x_np)
    inv = torch.empty_like(x)
    binding.slicemoe_permute_columns(cfg, x, inv, perm, inverse=True)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(tensors.to_numpy_f32(inv), oracle.permute_columns(x_np, perm_np, inverse=True))
    with pytest.raises(binding.SliceMoEError):
        binding.slicemoe_permute_columns(cfg, x, x, perm)


@pytest.mark.gpu
@pytest.mark.parametrize("name", ["bf16_tensor_core", "f32"])
def test_gpu_shuffled_slices_forward(name):
    import torch
    from paper_2510_04286_b200 import binding, tensors
    lc = GPU_SHAPES[name]
    h_np, w_np = synth.make_layer_inputs(lc, 2)
    perm_np = np.random.default_rng(5).permutation(lc.d).astype(np.int32)
    gpu = pu.GpuLayer(lc, h_np, w_np)
    perm = torch.from_numpy(perm_np).cuda()
    plain_h = gpu.h
    shuffled = torch.empty_like(plain_h)
    binding.slicemoe_permute_columns(gpu.cfg, plain_h, shuffled, perm)
    gpu.h = shuffled
    out_s, assigned, kept, idx, p = gpu.forward()
    out = torch.empty_like(out_s)
    binding.slicemoe_permute_columns(gpu.cfg, out_s, out, perm, inverse=True)
    torch.cuda.synchronize()
    assert gpu.status() == 0
    ocfg = pu.oracle_config(lc)
    idx_np = idx.cpu().numpy()
    free = oracle.forward_shuffled(ocfg, h_np, w_np, perm_np)
    pu.check_routing(free["probs"], free["gap"], free["topk_idx"], idx_np, p.cpu().numpy().astype(np.float64))
    ref = oracle.forward_shuffled(ocfg, h_np, w_np, perm_np, forced_idx=idx_np)["h_out"]
    pu.assert_outputs_close(tensors.to_numpy_f32(out), ref, lc.dtype)
    # and it is not the plain layer
    plain = oracle.forward(ocfg, h_np, w_np)["h_out"]
    assert np.abs(plain - ref).max() > 1e-3
