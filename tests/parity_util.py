"""GPU-vs-oracle comparison protocol shared by the GPU tests and the smoke check.

Routing: on every row whose oracle gap p_(k) - p_(k+1) exceeds GAP_TOL the GPU's set of k
experts must equal the oracle's; on the other rows (near-ties) each GPU-chosen expert must be
within GAP_TOL of the k-th oracle probability.  The number of such excluded rows is reported.
Everything downstream (counts, kept, offsets, dest, perm, stacked rows, expert outputs, h') is
then compared with the oracle re-run on the GPU's validated expert ids, so every element is
graded even where a near-tie was resolved differently.
"""
from __future__ import annotations

import numpy as np

import oracle
from paper_2510_04286_b200 import binding, synth, tensors

GAP_TOL = 1e-4
# bf16 storage: relative Frobenius error and elementwise error relative to rms(h'_oracle)
BF16_FRO, BF16_ELEM = 1e-2, 5e-2
# fp32 storage: elementwise error relative to max(1, rms(h'_oracle))
F32_ELEM = 1e-4


def oracle_config(lc: synth.LayerConfig) -> oracle.OracleConfig:
    return oracle.OracleConfig(T=lc.T, d=lc.d, S=lc.S, E=lc.E, k=lc.k, Hr=lc.Hr, F=lc.F, act=lc.act,
                               capacity=lc.capacity, temperature=lc.temperature,
                               noise_sigma=lc.noise_sigma, noise_seed=lc.noise_seed)


def check_routing(probs, gap, ref_idx, gpu_idx, gpu_p=None):
    """Returns the number of excluded (near-tie) rows; raises AssertionError on a real mismatch."""
    N, k = gpu_idx.shape
    E = probs.shape[1]
    assert gpu_idx.min() >= 0 and gpu_idx.max() < E, "expert id out of range"
    srt = np.sort(gpu_idx, axis=1)
    assert np.all(srt[:, 1:] != srt[:, :-1]) if k > 1 else True, "an expert was chosen twice for a row"
    same_set = np.all(np.sort(ref_idx, axis=1) == srt, axis=1)
    clear = gap > GAP_TOL
    bad = clear & ~same_set
    assert not bad.any(), f"{bad.sum()} rows with a clear gap picked other experts, first row {np.argmax(bad)}"
    p_gpu_choice = np.take_along_axis(probs, gpu_idx.astype(np.int64), axis=1)
    p_kth = np.take_along_axis(probs, ref_idx[:, -1:].astype(np.int64), axis=1)
    near = ~clear
    ok = p_gpu_choice[near] >= p_kth[near] - GAP_TOL
    assert ok.all(), "a near-tie row picked an expert that is not within the tolerance of the k-th"
    if gpu_p is not None:
        err = np.abs(gpu_p - p_gpu_choice).max() if N else 0.0
        assert err <= 2e-4, f"gate probabilities differ from the oracle's by {err}"
        assert np.all(np.diff(gpu_p, axis=1) <= 1e-6), "top-k not listed most probable first"
    return int(near.sum())


def output_errors(got, ref):
    """(relative Frobenius, max |diff| / rms(ref), max |diff|, rms(ref)).  The rms is taken over
    the rows that received at least one expert output: rows whose pairs were all dropped by the
    capacity are exact zeros and would only deflate the scale."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    if ref.size == 0:
        return 0.0, 0.0, 0.0, 0.0
    diff = got - ref
    fro_ref = np.linalg.norm(ref)
    live = ref.reshape(ref.shape[0], -1).any(axis=1).sum() * (ref.size // max(ref.shape[0], 1))
    rms = fro_ref / np.sqrt(max(live, 1))
    fro = np.linalg.norm(diff) / fro_ref if fro_ref > 0 else np.linalg.norm(diff)
    mx = np.abs(diff).max()
    return float(fro), float(mx / rms) if rms > 0 else float(mx), float(mx), float(rms)


def assert_outputs_close(got, ref, dtype: str, what="h_out", one_ulp_of_element=False):
    """``one_ulp_of_element`` (the randomised shapes only; the named workloads are graded with the plain
    bound): the elementwise bound becomes 0.08 rms + 2^-7 |ref element| (one bf16 ulp of the element).
    Outputs whose largest elements are many times their rms (He-uniform weights with biases) miss the
    plain 0.05 rms even when the exact result is merely rounded to bf16 (0.025-0.04 of rms on such
    shapes against 0.013 on cfg1), and GELU units with z in [-4, -2] lose their last bits in
    1 + tanh (the activation runs in packed bf16): the forward measures up to 0.07 of rms on such
    shapes against 0.03 on cfg1, at a relative Frobenius error that stays at 3-5e-3 everywhere."""
    fro, rel_elem, mx, rms = output_errors(got, ref)
    if dtype == "bf16":
        assert fro <= BF16_FRO, f"{what}: relative Frobenius error {fro:.3e} > {BF16_FRO}"
        if one_ulp_of_element:
            diff = np.abs(np.asarray(got, np.float64) - np.asarray(ref, np.float64))
            bound = BF16_ELEM * rms + np.abs(np.asarray(ref, np.float64)) / 128.0
            worst = float((diff - bound).max()) if diff.size else 0.0
            assert worst <= 0.0, f"{what}: an element is {worst:.3e} past 0.05 rms + one bf16 ulp (rms {rms:.3e})"
        else:
            assert rel_elem <= BF16_ELEM, f"{what}: elementwise error {mx:.3e} is {rel_elem:.3e} of rms {rms:.3e}"
    else:
        assert mx <= F32_ELEM * max(1.0, rms), f"{what}: max |diff| {mx:.3e} (rms {rms:.3e})"
    return dict(rel_fro=fro, max_over_rms=rel_elem, max_abs=mx, rms=rms)


class GpuLayer:
    """Device tensors of one workload plus the calls through the C ABI."""

    def __init__(self, lc: synth.LayerConfig, h_np, w_np, device="cuda", drop_zero_biases=False):
        import torch
        self.torch = torch
        self.lc = lc
        self.cfg = tensors.config_from_synth(lc)
        self.dev = device
        self.h = tensors.to_torch(h_np, lc.dtype, device)
        self.w = tensors.weights_to_torch(w_np, lc.dtype, device, drop_zero_biases=drop_zero_biases)
        self.ws = binding.alloc_workspace(self.cfg, device)
        self.tdtype = binding.torch_dtype(self.cfg)

    def empty(self, shape, dtype):
        return self.torch.empty(shape, dtype=dtype, device=self.dev)

    def route(self, want_probs=True):
        t, c = self.torch, self.cfg
        idx = self.empty((c.N, c.k), t.int32)
        p = self.empty((c.N, c.k), t.float32)
        assigned = self.empty((c.E,), t.int32)
        probs = self.empty((c.N, c.E), t.float32) if want_probs else None
        binding.slicemoe_route(c, self.w, self.h, idx, p, assigned, probs, self.ws)
        return idx, p, assigned, probs

    def dispatch(self, idx, p):
        t, c = self.torch, self.cfg
        kept = self.empty((c.E,), t.int32)
        offsets = self.empty((c.E + 1,), t.int32)
        dest = self.empty((c.N, c.k), t.int32)
        perm = t.full((max(c.R, 1),), -1, dtype=t.int32, device=self.dev)
        xperm = t.zeros((max(c.R, 1), c.ds), dtype=self.tdtype, device=self.dev)
        binding.slicemoe_dispatch(c, self.h, idx, p, kept, offsets, dest, perm, xperm, self.ws)
        return kept, offsets, dest, perm, xperm

    def expert_ffn(self, xperm, offsets):
        c = self.cfg
        yperm = self.torch.zeros((max(c.R, 1), c.ds), dtype=self.tdtype, device=self.dev)
        binding.slicemoe_expert_ffn(c, self.w, xperm, offsets, yperm, self.ws)
        return yperm

    def combine(self, yperm, dest):
        c = self.cfg
        h_out = self.empty((c.T, c.d), self.tdtype)
        binding.slicemoe_combine(c, yperm, dest, h_out)
        return h_out

    def forward(self):
        t, c = self.torch, self.cfg
        h_out = self.empty((c.T, c.d), self.tdtype)
        assigned = self.empty((c.E,), t.int32)
        kept = self.empty((c.E,), t.int32)
        idx = self.empty((c.N, c.k), t.int32)
        p = self.empty((c.N, c.k), t.float32)
        binding.slicemoe_forward(c, self.w, self.h, h_out, self.ws, assigned, kept, idx, p)
        return h_out, assigned, kept, idx, p

    def status(self):
        return binding.slicemoe_last_status(self.ws)


def check_forward_against_oracle(lc: synth.LayerConfig, seed=0, sample_rows=None, rng_seed=0,
                                 one_ulp_of_element=False):
    """The whole protocol for the fused forward call.  With ``sample_rows`` only that many rows of
    h' are graded (chosen with a seeded generator), one by one; routing is always graded on all
    rows.  Returns a report dict."""
    import torch
    h_np, w_np = synth.make_layer_inputs(lc, seed)
    ocfg = oracle_config(lc)
    gpu = GpuLayer(lc, h_np, w_np)
    h_out, assigned, kept, idx, p = gpu.forward()
    torch.cuda.synchronize()
    assert gpu.status() == 0, f"device status {gpu.status()}"
    idx_np = idx.cpu().numpy()
    p_np = p.cpu().numpy().astype(np.float64)
    ref_route = oracle.route(ocfg, h_np, w_np)
    excluded = check_routing(ref_route["probs"], ref_route["gap"], ref_route["topk_idx"], idx_np, p_np)
    disp = oracle.dispatch(ocfg, idx_np)
    assert np.array_equal(assigned.cpu().numpy(), disp["assigned"]), "assigned counts differ"
    assert np.array_equal(kept.cpu().numpy(), disp["kept"]), "kept counts differ"
    got = tensors.to_numpy_f32(h_out).reshape(lc.N, lc.ds)
    dropped_rows = ~(disp["dest"] >= 0).any(axis=1)
    assert not got[dropped_rows].any(), "a row whose pairs were all dropped is not zero"
    if sample_rows is None or sample_rows >= lc.N:
        ref = oracle.forward(ocfg, h_np, w_np, forced_idx=idx_np)["h_out"].reshape(lc.N, lc.ds)
        errs = assert_outputs_close(got, ref, lc.dtype, one_ulp_of_element=one_ulp_of_element)
    else:
        # seeded random rows plus the first rows (under a capacity the kept pairs sit at the front)
        pick = np.random.default_rng(rng_seed).choice(lc.N, sample_rows, replace=False)
        pick = np.unique(np.concatenate([pick, np.arange(min(lc.N, 1024))]))
        ref = oracle.rows(ocfg, h_np, w_np, pick, idx_np[pick], disp["dest"][pick] >= 0)["y"]
        errs = assert_outputs_close(got[pick], ref, lc.dtype, one_ulp_of_element=one_ulp_of_element)
    drift = int(np.abs(disp["assigned"] - ref_route["assigned"]).sum())
    assert drift <= 2 * excluded, "assigned counts drift from the free oracle by more than the near-ties allow"
    return dict(excluded=excluded, rows=lc.N, **errs)
