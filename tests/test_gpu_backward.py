"""GPU parity of slicemoe_backward against the oracle's backward (Section 3.1: the layer is trained
end to end; gradients by the chain rule on the forward of Section 3.1 / Eq. 1).

The GPU forward supplies the expert ids and gates; the oracle differentiates the same function on
those ids (forced routing), so near-ties in the router cannot make the two sides differ.  The kernels
compute in fp32 on the stored values, so every gradient is held to a relative Frobenius error of 1e-4
(fp32 sums of up to a few thousand terms in an order that differs from the oracle's) and, element by
element, to 1e-4 * max(1, rms); dL/dh of a bf16 layer is rounded to bf16 once on output, which alone
is 2^-9 per element, hence 4e-3 there."""
from dataclasses import replace

import numpy as np
import pytest

import oracle
from paper_2510_04286_b200 import binding, synth

import parity_util as pu

pytestmark = pytest.mark.gpu

GRADS = ("dWr1", "dbr1", "dWr2", "dbr2", "dW1", "db1", "dW2", "db2")
F32_FRO, BF16_DH_FRO, ELEM = 1e-4, 4e-3, 1e-4


def run_backward(lc, seed=0, with_bias_grads=True, accumulate_twice=False, drop_zero_biases=False):
    import torch
    h, w = synth.make_layer_inputs(lc, seed)
    gout = synth.make_grad_out(lc, seed)
    gpu = pu.GpuLayer(lc, h, w, drop_zero_biases=drop_zero_biases)
    c = gpu.cfg
    _, _, _, idx, p = gpu.forward()
    g_dev = pu.tensors.to_torch(gout, lc.dtype, "cuda")
    shapes = dict(dWr1=(c.Hr, c.ds), dbr1=(c.Hr,), dWr2=(c.E, c.Hr), dbr2=(c.E,), dW1=(c.E, c.F, c.ds),
                  db1=(c.E, c.F), dW2=(c.E, c.ds, c.F), db2=(c.E, c.ds))
    grads = {n: torch.full(s, 7.0, dtype=torch.float32, device="cuda") for n, s in shapes.items()
             if with_bias_grads or not n.startswith("db")}
    dh = torch.full((c.T, c.d), 3.0, dtype=gpu.tdtype, device="cuda")
    ws = torch.empty(binding.slicemoe_backward_workspace_bytes(c), dtype=torch.uint8, device="cuda")
    binding.slicemoe_backward(c, gpu.w, gpu.h, g_dev, idx, p, dh, grads, ws)
    if accumulate_twice:
        binding.slicemoe_backward(c, gpu.w, gpu.h, g_dev, idx, p, dh, grads, ws, accumulate=True)
    torch.cuda.synchronize()
    ref = oracle.backward(pu.oracle_config(lc), h, w, gout, forced_idx=idx.cpu().numpy())
    got = {n: t.cpu().numpy().astype(np.float64) for n, t in grads.items()}
    got["dh"] = pu.tensors.to_numpy_f32(dh).astype(np.float64)
    return got, ref


def compare(got, ref, lc, scale=1.0):
    report = {}
    for name, g in got.items():
        r = ref[name] * scale
        norm = np.linalg.norm(r)
        fro = np.linalg.norm(g - r) / norm if norm > 0 else np.linalg.norm(g - r)
        rms = norm / np.sqrt(max(r.size, 1))
        mx = np.abs(g - r).max() if r.size else 0.0
        bf16_dh = name == "dh" and lc.dtype == "bf16"
        assert fro <= (BF16_DH_FRO if bf16_dh else F32_FRO), f"{name}: relative Frobenius error {fro:.3e}"
        if bf16_dh:
            assert np.all(np.abs(g - r) <= 2.0 ** -8 * np.abs(r) + ELEM * max(1.0, rms)), f"{name}: element off"
        else:
            assert mx <= ELEM * max(1.0, rms), f"{name}: max |diff| {mx:.3e} (rms {rms:.3e})"
        report[name] = fro
    return report


CASES = {
    "cfg0_fp32_relu_biases": synth.CONFIGS["cfg0"],
    "cfg1_ragged": synth.CONFIGS["cfg1"].with_tokens(301),
    "cfg2_E32": synth.CONFIGS["cfg2"].with_tokens(70),
    "cfg3b_capacity_wide_rows": synth.CONFIGS["cfg3b"].with_tokens(96),
    "cfg4_decode": synth.CONFIGS["cfg4"].with_tokens(24),
    "paper768_k3": synth.CONFIGS["paper768_k3"].with_tokens(50),
    "paper768_S32_narrow": synth.CONFIGS["paper768_S32"].with_tokens(20),
    "temperature": replace(synth.CONFIGS["cfg1"].with_tokens(64), temperature=2.0),
    "fp32_gelu_k1": replace(synth.CONFIGS["cfg0"], T=100, act=synth.ACT_GELU_TANH, k=1),
    "logit_noise": replace(synth.CONFIGS["cfg1"].with_tokens(64), noise_sigma=0.5, noise_seed=7, temperature=0.7),
}


@pytest.mark.parametrize("name", list(CASES))
def test_backward_matches_oracle(name):
    lc = CASES[name]
    got, ref = run_backward(lc)
    if lc.capacity:
        assert np.abs(ref["dh"].reshape(lc.N, lc.ds)).max(axis=1).min() == 0.0, "no slice was dropped"
    compare(got, ref, lc)


def test_bias_gradients_optional_and_accumulation():
    lc = synth.CONFIGS["cfg0"].with_tokens(64)
    got, ref = run_backward(lc, with_bias_grads=False)
    assert set(got) == {"dh", "dWr1", "dWr2", "dW1", "dW2"}
    compare(got, ref, lc)
    got2, ref2 = run_backward(lc, accumulate_twice=True)
    dh = got2.pop("dh")
    compare(got2, ref2, lc, scale=2.0)          # the second call added to the first
    compare(dict(dh=dh), ref2, lc)              # dL/dh is overwritten, not accumulated


def test_backward_is_deterministic_in_dh_and_stable_in_weights():
    lc = synth.CONFIGS["cfg1"].with_tokens(200)
    a, _ = run_backward(lc)
    b, _ = run_backward(lc)
    assert np.array_equal(a["dh"], b["dh"])
    for n in GRADS:
        assert np.allclose(a[n], b[n], rtol=1e-4, atol=1e-6)


def test_backward_rejects_bad_arguments():
    import torch
    lc = synth.CONFIGS["cfg0"].with_tokens(16)
    c = pu.tensors.config_from_synth(lc)
    with pytest.raises(binding.SliceMoEError) as e:      # slices too wide for the kernels' tiles
        binding.slicemoe_backward_workspace_bytes(binding.Config(T=8, d=4096, S=1, E=4, k=1, F=64))
    assert e.value.status == 3
    h, w = synth.make_layer_inputs(lc, 0)
    gpu = pu.GpuLayer(lc, h, w)
    _, _, _, idx, p = gpu.forward()
    grads = dict(dWr1=torch.zeros(c.Hr, c.ds, device="cuda"), dWr2=torch.zeros(c.E, c.Hr, device="cuda"),
                 dW1=torch.zeros(c.E, c.F, c.ds, device="cuda"), dW2=torch.zeros(c.E, c.ds, c.F, device="cuda"))
    ws = torch.empty(binding.slicemoe_backward_workspace_bytes(c), dtype=torch.uint8, device="cuda")
    dh = torch.empty_like(gpu.h)
    with pytest.raises(binding.SliceMoEError) as e:      # grad_h aliases h
        binding.slicemoe_backward(c, gpu.w, gpu.h, dh, idx, p, gpu.h, grads, ws)
    assert e.value.status == 6
    with pytest.raises(binding.SliceMoEError) as e:      # workspace too small
        binding.slicemoe_backward(c, gpu.w, gpu.h, dh, idx, p, dh.clone(), grads, ws[:256])
    assert e.value.status == 5
    with pytest.raises(binding.SliceMoEError) as e:      # a weight gradient is missing
        binding.slicemoe_backward(c, gpu.w, gpu.h, dh, idx, p, dh.clone(), dict(grads, dW1=None), ws)
    assert e.value.status == 1


def test_backward_of_an_empty_batch():
    import torch
    lc = synth.CONFIGS["cfg0"].with_tokens(0)
    c = pu.tensors.config_from_synth(lc)
    _, w = synth.make_layer_inputs(lc, 0)
    wd = pu.tensors.weights_to_torch(w, lc.dtype, "cuda")
    grads = dict(dWr1=torch.ones(c.Hr, c.ds, device="cuda"), dWr2=torch.ones(c.E, c.Hr, device="cuda"),
                 dW1=torch.ones(c.E, c.F, c.ds, device="cuda"), dW2=torch.ones(c.E, c.ds, c.F, device="cuda"))
    ws = torch.empty(max(binding.slicemoe_backward_workspace_bytes(c), 256), dtype=torch.uint8, device="cuda")
    e = torch.empty((0, c.d), device="cuda")   # empty tensors carry no address
    idx = torch.empty((0, c.k), dtype=torch.int32, device="cuda")
    p = torch.empty((0, c.k), dtype=torch.float32, device="cuda")
    binding.slicemoe_backward(c, wd, e, e, idx, p, e, grads, ws)
    torch.cuda.synchronize()
    assert all(float(t.abs().max()) == 0.0 for t in grads.values())


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3b"])
def test_backward_full_size_sampled_rows_and_invariants(name):
    """The named workloads at their full size, as bench.py launches them.  dL/dh of a kept slice depends
    on that slice alone, so sampled slices are graded against the oracle run on just those slices as an
    S = 1 layer of width ds (the reshape equivalence the forward oracle is pinned to) with the GPU's
    expert ids; slices dropped by the capacity must come out as exact zeros.  The weight gradients, sums
    over all slices, are checked through what the mathematics fixes: db2 is the per-expert sum of grad_out
    over the kept pairs, the logit gradients of every row sum to zero (so dbr2 and the columns of dWr2 do);
    without a capacity the weight gradients of a 2048-token prefix alone are compared with the oracle's."""
    import torch
    lc = synth.CONFIGS[name]
    h, w = synth.make_layer_inputs(lc, 0)
    gout = synth.make_grad_out(lc, 0)
    gpu = pu.GpuLayer(lc, h, w)
    c = gpu.cfg
    _, _, _, idx, p = gpu.forward()
    g_dev = pu.tensors.to_torch(gout, lc.dtype, "cuda")
    shapes = dict(dWr1=(c.Hr, c.ds), dbr1=(c.Hr,), dWr2=(c.E, c.Hr), dbr2=(c.E,), dW1=(c.E, c.F, c.ds),
                  db1=(c.E, c.F), dW2=(c.E, c.ds, c.F), db2=(c.E, c.ds))
    grads = {n: torch.empty(s, dtype=torch.float32, device="cuda") for n, s in shapes.items()}
    dh = torch.empty((c.T, c.d), dtype=gpu.tdtype, device="cuda")
    ws = torch.empty(binding.slicemoe_backward_workspace_bytes(c), dtype=torch.uint8, device="cuda")
    binding.slicemoe_backward(c, gpu.w, gpu.h, g_dev, idx, p, dh, grads, ws)
    torch.cuda.synchronize()
    idx_np = idx.cpu().numpy()
    got = {n: t.cpu().numpy().astype(np.float64) for n, t in grads.items()}
    dX = pu.tensors.to_numpy_f32(dh).astype(np.float64).reshape(lc.N, lc.ds)
    X, G = h.reshape(lc.N, lc.ds), gout.reshape(lc.N, lc.ds)
    kept = oracle.dispatch(pu.oracle_config(lc), idx_np)["dest"] >= 0            # [N, k]

    # sampled slices whose pairs were all kept (first, last and a seeded draw)
    rng = np.random.default_rng(7)
    cand = np.flatnonzero(kept.all(axis=1))
    rows = np.unique(np.concatenate([cand[:1], cand[-1:], rng.choice(cand, 2046)]))
    sub = replace(lc, T=len(rows), d=lc.ds, S=1, capacity=0)
    ref = oracle.backward(pu.oracle_config(sub), X[rows], w, G[rows], forced_idx=idx_np[rows])
    compare(dict(dh=dX[rows]), ref, sub)
    if lc.capacity:
        gone = ~kept.any(axis=1)
        assert gone.any() and np.abs(dX[gone]).max() == 0.0

    # db2[e] = sum of grad_out over the pairs kept on e
    db2 = np.zeros((lc.E, lc.ds))
    for j in range(lc.k):
        np.add.at(db2, idx_np[kept[:, j], j], G[kept[:, j]].astype(np.float64))
    compare(dict(db2=got["db2"]), dict(db2=db2), lc)
    scale = np.abs(got["dbr2"]).max()
    assert scale > 0 and abs(got["dbr2"].sum()) <= 1e-4 * scale * lc.E
    assert np.abs(got["dWr2"].sum(axis=0)).max() <= 1e-4 * np.abs(got["dWr2"]).max() * lc.E

    if not lc.capacity and name == "cfg1":
        # weight gradients of a 2048-token prefix against the oracle (the generator's prefix property)
        pre = lc.with_tokens(2048)
        binding.slicemoe_backward(pu.tensors.config_from_synth(pre), gpu.w, gpu.h[:2048], g_dev[:2048],
                                  idx[:pre.N], p[:pre.N], dh[:2048], grads, ws)
        torch.cuda.synchronize()
        ref = oracle.backward(pu.oracle_config(pre), h[:2048], w, gout[:2048], forced_idx=idx_np[:pre.N])
        compare({n: t.cpu().numpy().astype(np.float64) for n, t in grads.items()}, ref, pre)


@pytest.mark.parametrize("name,rate", [("cfg0", 0.2), ("cfg1", 0.5), ("paper768_k3", 0.5), ("cfg1", 0.0)])
def test_train_mode_backward_with_dropout_gates(name, rate):
    """Section 3.3 inside the backward: route -> slicemoe_gate_dropout -> slicemoe_backward with
    dropout_gates, against the oracle's backward on the same expert ids and the oracle's own mask (the
    masks of the two sides agree bit for bit: an integer compare of the same Philox word)."""
    import torch
    lc = synth.CONFIGS[name].with_tokens(120)
    h, w = synth.make_layer_inputs(lc, 0)
    gout = synth.make_grad_out(lc, 0)
    gpu = pu.GpuLayer(lc, h, w)
    c = gpu.cfg
    idx, p, _, _ = gpu.route(want_probs=False)
    p_plain = p.cpu().numpy().astype(np.float64)
    binding.slicemoe_gate_dropout(c, p, 1234, rate)
    _, dropped = oracle.gate_dropout(p_plain, 1234, rate)
    gates = p.cpu().numpy()
    assert np.array_equal(gates == 0.0, dropped & ~(dropped.all(axis=1, keepdims=True) & (np.arange(lc.k) == 0)))
    g_dev = pu.tensors.to_torch(gout, lc.dtype, "cuda")
    shapes = dict(dWr1=(c.Hr, c.ds), dbr1=(c.Hr,), dWr2=(c.E, c.Hr), dbr2=(c.E,), dW1=(c.E, c.F, c.ds),
                  db1=(c.E, c.F), dW2=(c.E, c.ds, c.F), db2=(c.E, c.ds))
    grads = {n: torch.empty(s, dtype=torch.float32, device="cuda") for n, s in shapes.items()}
    dh = torch.empty((c.T, c.d), dtype=gpu.tdtype, device="cuda")
    ws = torch.empty(binding.slicemoe_backward_workspace_bytes(c), dtype=torch.uint8, device="cuda")
    binding.slicemoe_backward(c, gpu.w, gpu.h, g_dev, idx, p, dh, grads, ws, dropout_gates=True)
    torch.cuda.synchronize()
    ref = oracle.backward(pu.oracle_config(lc), h, w, gout, forced_idx=idx.cpu().numpy(), dropped=dropped)
    got = {n: t.cpu().numpy().astype(np.float64) for n, t in grads.items()}
    got["dh"] = pu.tensors.to_numpy_f32(dh).astype(np.float64)
    compare(got, ref, lc)
    if rate > 0:
        assert dropped.any()


@pytest.mark.parametrize("name,rate", [("cfg1", 0.2), ("cfg4", 0.3), ("cfg0", 0.2)])
def test_training_step_forward_train_mode_then_backward(name, rate):
    """A whole training step through the library: slicemoe_forward with cfg.train_gates (the gates drawn inside
    the forward: in the one-launch kernel for 64-wide slices, by the gate step of the stage-by-stage forms
    otherwise) hands its ids and gates to slicemoe_backward with dropout_gates; graded against the oracle's
    backward on the same ids with the oracle's own mask."""
    import dataclasses
    import torch
    lc = synth.CONFIGS[name].with_tokens(120 if name != "cfg4" else 32)
    h, w = synth.make_layer_inputs(lc, 0)
    gout = synth.make_grad_out(lc, 0)
    gpu = pu.GpuLayer(lc, h, w)
    p_plain = gpu.forward()[4].cpu().numpy().astype(np.float64)
    gpu.cfg = dataclasses.replace(gpu.cfg, train_gates=1, dropout_rate=rate, dropout_seed=99)
    c = gpu.cfg
    _, _, _, idx, gates = gpu.forward()
    torch.cuda.synchronize()
    _, dropped = oracle.gate_dropout(p_plain, 99, rate)
    assert np.array_equal(gates.cpu().numpy() == 0.0,
                          dropped & ~(dropped.all(axis=1, keepdims=True) & (np.arange(lc.k) == 0)))
    assert dropped.any()
    g_dev = pu.tensors.to_torch(gout, lc.dtype, "cuda")
    shapes = dict(dWr1=(c.Hr, c.ds), dbr1=(c.Hr,), dWr2=(c.E, c.Hr), dbr2=(c.E,), dW1=(c.E, c.F, c.ds),
                  db1=(c.E, c.F), dW2=(c.E, c.ds, c.F), db2=(c.E, c.ds))
    grads = {n: torch.empty(s_, dtype=torch.float32, device="cuda") for n, s_ in shapes.items()}
    dh = torch.empty((c.T, c.d), dtype=gpu.tdtype, device="cuda")
    ws = torch.empty(binding.slicemoe_backward_workspace_bytes(c), dtype=torch.uint8, device="cuda")
    binding.slicemoe_backward(c, gpu.w, gpu.h, g_dev, idx, gates, dh, grads, ws, dropout_gates=True)
    torch.cuda.synchronize()
    ref = oracle.backward(pu.oracle_config(lc), h, w, gout, forced_idx=idx.cpu().numpy(), dropped=dropped)
    got = {n: t.cpu().numpy().astype(np.float64) for n, t in grads.items()}
    got["dh"] = pu.tensors.to_numpy_f32(dh).astype(np.float64)
    compare(got, ref, lc)


@pytest.mark.parametrize("block", range(3))
def test_backward_random_shapes(block):
    """Seeded random shapes: widths inside and outside the tensor-core set, fp32 and bf16 storage,
    expert counts that are not multiples of four, hidden widths that end in a partial chunk, k = 1..4,
    ragged token counts, capacities, both activations, NULL bias pointers."""
    import random
    rnd = random.Random(2000 + block)
    for it in range(8):
        dtype = rnd.choice(["bf16", "bf16", "f32"])
        V = 8 if dtype == "bf16" else 4
        ds = rnd.choice([8, 24, 40, 64, 96, 128, 200, 256, 384])
        ds -= ds % V
        S = rnd.choice([1, 2, 4])
        E = rnd.choice([3, 5, 8, 16, 21, 64])
        k = min(E, rnd.choice([1, 2, 2, 3, 4]))
        T = rnd.choice([1, 7, 33, 100, 250])
        cap = max(1, int(rnd.uniform(0.3, 1.5) * T * S * k / E)) if rnd.random() < 0.3 else 0
        lc = synth.LayerConfig(f"bwd_rand{block}_{it}", T=T, d=ds * S, S=S, E=E, k=k, F=V * rnd.randint(2, 70),
                               Hr=V * rnd.choice([4, 16, 32, 40]), dtype=dtype, act=rnd.choice([0, 1]),
                               init=rnd.choice(["normal", "kaiming"]), capacity=cap,
                               wr2_gain=rnd.choice([1.0, 30.0]))
        try:
            got, ref = run_backward(lc, seed=it, drop_zero_biases=rnd.random() < 0.5)
            compare(got, ref, lc)
        except AssertionError as ex:
            raise AssertionError(f"{lc}: {ex}") from ex


def test_backward_ignores_expert_ids_outside_the_layer():
    """An id outside [0, E) in topk_idx (never produced by the forward) is treated as not routed: the
    other rows' dL/dh are bit-identical and nothing is read or written out of range."""
    import torch
    lc = synth.CONFIGS["cfg1"].with_tokens(40)
    h, w = synth.make_layer_inputs(lc, 0)
    gpu = pu.GpuLayer(lc, h, w)
    c = gpu.cfg
    _, _, _, idx, p = gpu.forward()
    g_dev = pu.tensors.to_torch(synth.make_grad_out(lc, 0), lc.dtype, "cuda")
    grads = dict(dWr1=torch.empty(c.Hr, c.ds, device="cuda"), dWr2=torch.empty(c.E, c.Hr, device="cuda"),
                 dW1=torch.empty(c.E, c.F, c.ds, device="cuda"), dW2=torch.empty(c.E, c.ds, c.F, device="cuda"))
    ws = torch.empty(binding.slicemoe_backward_workspace_bytes(c), dtype=torch.uint8, device="cuda")
    dh_ok, dh_bad = torch.empty_like(gpu.h), torch.empty_like(gpu.h)
    binding.slicemoe_backward(c, gpu.w, gpu.h, g_dev, idx, p, dh_ok, grads, ws)
    bad = idx.clone()
    bad[5, 0] = c.E + 3
    bad[9, 1] = -2
    for mode in (False, True):
        binding.slicemoe_backward(c, gpu.w, gpu.h, g_dev, bad, p, dh_bad, grads, ws, dropout_gates=mode)
        torch.cuda.synchronize()
        assert all(bool(torch.isfinite(t).all()) for t in grads.values())
        if not mode:
            rows_ok = torch.ones(c.N, dtype=torch.bool, device="cuda")
            rows_ok[5] = rows_ok[9] = False
            a = dh_ok.reshape(c.N, c.ds)[rows_ok]
            b = dh_bad.reshape(c.N, c.ds)[rows_ok]
            assert torch.equal(a, b)


def test_backward_through_shuffled_slices():
    """Figure 5's shuffled layer: slicemoe_permute_columns around the forward and, for the gradient, around
    slicemoe_backward (dL/dh = P^-1 backward(P h, P grad_out)); against the same composition of oracle calls."""
    import torch
    lc = synth.CONFIGS["cfg1"].with_tokens(90)
    h, w = synth.make_layer_inputs(lc, 3)
    gout = synth.make_grad_out(lc, 3)
    perm_np = np.random.default_rng(5).permutation(lc.d).astype(np.int32)
    gpu = pu.GpuLayer(lc, h, w)
    c = gpu.cfg
    perm = torch.from_numpy(perm_np).cuda()
    g_dev = pu.tensors.to_torch(gout, lc.dtype, "cuda")
    h_s, g_s = torch.empty_like(gpu.h), torch.empty_like(g_dev)
    binding.slicemoe_permute_columns(c, gpu.h, h_s, perm)
    binding.slicemoe_permute_columns(c, g_dev, g_s, perm)
    gpu.h = h_s
    _, _, _, idx, p = gpu.forward()
    grads = dict(dWr1=torch.empty(c.Hr, c.ds, device="cuda"), dWr2=torch.empty(c.E, c.Hr, device="cuda"),
                 dW1=torch.empty(c.E, c.F, c.ds, device="cuda"), dW2=torch.empty(c.E, c.ds, c.F, device="cuda"))
    ws = torch.empty(binding.slicemoe_backward_workspace_bytes(c), dtype=torch.uint8, device="cuda")
    dx, dh = torch.empty_like(h_s), torch.empty_like(h_s)
    binding.slicemoe_backward(c, gpu.w, h_s, g_s, idx, p, dx, grads, ws)
    binding.slicemoe_permute_columns(c, dx, dh, perm, inverse=True)
    torch.cuda.synchronize()
    ref = oracle.backward(pu.oracle_config(lc), oracle.permute_columns(h, perm_np), w,
                          oracle.permute_columns(gout, perm_np), forced_idx=idx.cpu().numpy())
    ref["dh"] = oracle.permute_columns(ref["dh"], perm_np, inverse=True)
    got = {n: t.cpu().numpy().astype(np.float64) for n, t in grads.items()}
    got["dh"] = pu.tensors.to_numpy_f32(dh).astype(np.float64)
    compare(got, ref, lc)
