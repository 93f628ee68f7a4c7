"""GPU parity: every C-ABI call against the fp64 oracle on the same seeded inputs."""
import dataclasses

import numpy as np
import pytest

import oracle
from paper_2510_04286_b200 import binding, synth, tensors

import parity_util as pu

pytestmark = pytest.mark.gpu

C = synth.CONFIGS
LC = synth.LayerConfig

# Small shapes that still span several row tiles, dispatch chunks and ragged tails.
SMALL = {
    "f32_tiny": C["cfg0"].with_tokens(77),
    "f32_cfg0": C["cfg0"],
    "bf16_lm": C["cfg1"].with_tokens(333),                       # N = 2664, R = 5328
    "bf16_wide": C["cfg2"].with_tokens(150),                     # N = 2400, E = 32
    "bf16_skew_cap": C["cfg3b"].with_tokens(96),                 # ds = 256, F = 1024, k = 1, capacity
    "bf16_skew_literal": C["cfg3"].with_tokens(64),              # everything to expert 0, most dropped
    "bf16_decode": C["cfg4"].with_tokens(16),                    # ds = 128, F = 512, E = 64
    "bf16_paper_slice96": LC("s96", T=40, d=768, S=8, E=16, k=2, F=384),   # the paper's own ds = 96
    "bf16_k3": LC("k3", T=50, d=256, S=4, E=8, k=3, F=256),
    "f32_gelu_cap": LC("f32cap", T=90, d=128, S=2, E=4, k=2, F=128, dtype="f32", capacity=50, init="kaiming"),
    "bf16_one_expert": LC("e1", T=20, d=128, S=2, E=1, k=1, F=256),
    "bf16_k_equals_E": LC("kE", T=20, d=128, S=2, E=2, k=2, F=256),
    "bf16_single_row": LC("one", T=1, d=64, S=1, E=16, k=2, F=256),
    # more of the tensor-core set: weights that stream through the rings (more chunks than slots),
    # ReLU experts, biases that are not zero, E = 64 at ds = 64, ds = 256 with k = 2
    "bf16_streamed": LC("stream", T=300, d=256, S=2, E=16, k=2, F=1024, Hr=512),
    "bf16_relu_biased": LC("relub", T=200, d=256, S=4, E=32, k=2, F=256, act=0, init="kaiming"),
    "bf16_gelu_biased": LC("gelub", T=130, d=512, S=4, E=16, k=1, F=512, init="kaiming"),
    "bf16_e64_ds64": LC("e64", T=260, d=128, S=2, E=64, k=2, F=128),
    "bf16_ds256_k2": LC("w256", T=70, d=512, S=2, E=16, k=2, F=512, Hr=128),
    # 256-wide slices, k = 1, few tiles: the expert pass runs every tile as two tiles over halves of the hidden layer
    # (W2's column halves, b2 added once); real biases
    "bf16_ds256_k1_split": LC("w256k1", T=300, d=512, S=2, E=16, k=1, F=512, init="kaiming"),
    # the paper's d = 768 at S = 16 and S = 4: 48- and 192-wide slices on zero-filled 64 / 256-wide tiles
    # eight experts on the 16-wide router instantiation (padded experts masked out)
    "bf16_e8": LC("e8", T=150, d=512, S=4, E=8, k=2, F=512),
    # k = 3 (the paper's Table 4) on the tensor-core kernels: stacked outputs + combine kernel
    "bf16_k3_tc": LC("k3tc", T=200, d=512, S=8, E=16, k=3, F=256),
    "bf16_k3_slice96": LC("k3s96", T=300, d=768, S=8, E=16, k=3, F=384),   # k = 3 at the paper's own width: four launches + combine
    "bf16_paper_slice48": LC("s48", T=50, d=768, S=16, E=16, k=2, F=192),
    "bf16_paper_slice192": LC("s192", T=60, d=768, S=4, E=16, k=2, F=768),
    # S = 2 and S = 32 of the same sweep: 384- and 24-wide slices, CUDA-core kernels
    "bf16_paper_slice384": LC("s384", T=40, d=768, S=2, E=16, k=2, F=1536),
    "bf16_paper_slice24": LC("s24", T=40, d=768, S=32, E=16, k=2, F=96),
}


def inputs(lc, seed=0):
    return synth.make_layer_inputs(lc, seed)


@pytest.mark.parametrize("name", list(SMALL))
def test_route(name):
    import torch
    lc = SMALL[name]
    h, w = inputs(lc)
    gpu = pu.GpuLayer(lc, h, w)
    idx, p, assigned, probs = gpu.route()
    torch.cuda.synchronize()
    ref = oracle.route(pu.oracle_config(lc), h, w)
    idx_np = idx.cpu().numpy()
    pu.check_routing(ref["probs"], ref["gap"], ref["topk_idx"], idx_np, p.cpu().numpy().astype(np.float64))
    assert np.abs(probs.cpu().numpy() - ref["probs"]).max() <= 2e-4
    np.testing.assert_array_equal(assigned.cpu().numpy(), np.bincount(idx_np.ravel(), minlength=lc.E))
    assert assigned.sum().item() == lc.R


@pytest.mark.parametrize("T,d,S,E,k,init", [
    (5000, 1024, 4, 64, 1, "normal"),     # 256-wide rows, 157 tiles: CTAs with two tiles and with one, ragged last tile
    (2500, 1024, 4, 64, 2, "normal"),     # 256-wide rows, 79 tiles on 79 CTAs, ragged last tile; k = 2
    (12000, 768, 4, 16, 2, "kaiming"),    # 192-wide rows (zero-filled fourth panel), three tiles per CTA, real biases
    (30000, 512, 4, 32, 2, "normal"),     # 128-wide rows: two panels, three row tiles in shared memory, 7 tiles per CTA
    (9000, 768, 8, 8, 1, "kaiming"),      # 96-wide rows (zero-filled second panel), E = 8 on the 16-wide instantiation
    (100, 256, 1, 16, 2, "normal"),       # one ragged tile
    (9000, 768, 8, 16, 3, "normal"),      # k = 3 (the paper's Table 4 shape): the third pick by repeated arg-max
    (3000, 1024, 4, 64, 5, "kaiming"),    # k = 5 of 64 experts on 256-wide rows
])
def test_route_resident_weights(T, d, S, E, k, init):
    """slicemoe_route without the probability matrix on slices of 96 to 256 elements (router hidden width 256):
    the router that keeps both weight matrices in shared memory.  Routing on every row, the returned
    probabilities and the per-expert counts against the oracle; the probability-matrix form (another kernel) must
    pick the same experts wherever the gap is clear."""
    import torch
    lc = LC(f"rw_T{T}_d{d}_S{S}_E{E}_k{k}_{init}", T=T, d=d, S=S, E=E, k=k, F=2 * (d // S), init=init)
    assert lc.Hr == 256 and lc.ds in (96, 128, 192, 256)
    h, w = inputs(lc)
    gpu = pu.GpuLayer(lc, h, w)
    idx, p, assigned, _ = gpu.route(want_probs=False)
    torch.cuda.synchronize()
    assert gpu.status() == 0
    ref = oracle.route(pu.oracle_config(lc), h, w)
    idx_np = idx.cpu().numpy()
    excluded = pu.check_routing(ref["probs"], ref["gap"], ref["topk_idx"], idx_np, p.cpu().numpy().astype(np.float64))
    np.testing.assert_array_equal(assigned.cpu().numpy(), np.bincount(idx_np.ravel(), minlength=lc.E))
    assert assigned.sum().item() == lc.R
    idx2, p2, _, _ = gpu.route(want_probs=True)
    torch.cuda.synchronize()
    clear = ref["gap"] > pu.GAP_TOL
    np.testing.assert_array_equal(np.sort(idx2.cpu().numpy(), axis=1)[clear], np.sort(idx_np, axis=1)[clear])
    again = gpu.route(want_probs=False)
    torch.cuda.synchronize()
    assert torch.equal(again[0], idx) and torch.equal(again[1], p) and torch.equal(again[2], assigned)
    print(lc.name, "excluded near-tie rows", excluded, "of", lc.N)


@pytest.mark.parametrize("name", list(SMALL))
def test_dispatch(name):
    import torch
    lc = SMALL[name]
    h, w = inputs(lc)
    gpu = pu.GpuLayer(lc, h, w)
    ocfg = pu.oracle_config(lc)
    # routing input: the oracle's own top-k (dispatch is graded on its own)
    ref_route = oracle.route(ocfg, h, w)
    idx = torch.from_numpy(ref_route["topk_idx"]).cuda()
    p = torch.from_numpy(ref_route["topk_p"].astype(np.float32)).cuda()
    kept, offsets, dest, perm, xperm = gpu.dispatch(idx, p)
    torch.cuda.synchronize()
    ref = oracle.dispatch(ocfg, ref_route["topk_idx"])
    np.testing.assert_array_equal(kept.cpu().numpy(), ref["kept"])
    np.testing.assert_array_equal(offsets.cpu().numpy(), ref["offsets"])
    np.testing.assert_array_equal(dest.cpu().numpy(), ref["dest"])
    n_kept = int(ref["offsets"][-1])
    np.testing.assert_array_equal(perm.cpu().numpy()[:n_kept], ref["perm"])
    assert np.all(perm.cpu().numpy()[n_kept:] == -1)            # nothing written past the kept rows
    want = oracle.weight_slices(ocfg, h, p.cpu().numpy().astype(np.float64), ref["dest"], n_kept)
    got = tensors.to_numpy_f32(xperm)[:n_kept]
    # Eq. 1 with one rounding to the storage type
    tol = 2.0 ** -8 if lc.dtype == "bf16" else 2.0 ** -23
    assert np.all(np.abs(got - want) <= tol * np.abs(want) + 1e-30)
    assert not tensors.to_numpy_f32(xperm)[n_kept:].any()


@pytest.mark.parametrize("name", list(SMALL))
def test_expert_ffn_and_combine(name):
    import torch
    lc = SMALL[name]
    h, w = inputs(lc)
    gpu = pu.GpuLayer(lc, h, w)
    ocfg = pu.oracle_config(lc)
    ref_route = oracle.route(ocfg, h, w)
    idx = torch.from_numpy(ref_route["topk_idx"]).cuda()
    p = torch.from_numpy(ref_route["topk_p"].astype(np.float32)).cuda()
    kept, offsets, dest, perm, xperm = gpu.dispatch(idx, p)
    yperm = gpu.expert_ffn(xperm, offsets)
    h_out = gpu.combine(yperm, dest)
    torch.cuda.synchronize()
    assert gpu.status() == 0
    n_kept = int(offsets[-1].item())
    x_in = tensors.to_numpy_f32(xperm)[:n_kept].astype(np.float64)
    want_y = oracle.expert_ffn(ocfg, x_in, offsets.cpu().numpy(), w)
    got_y = tensors.to_numpy_f32(yperm)
    pu.assert_outputs_close(got_y[:n_kept], want_y, lc.dtype, "yperm")
    assert not got_y[n_kept:].any()                               # rows past offsets[E] untouched
    want_h = oracle.combine(ocfg, got_y[:max(n_kept, 1)].astype(np.float64), dest.cpu().numpy())
    got_h = tensors.to_numpy_f32(h_out)
    tol = 2.0 ** -8 if lc.dtype == "bf16" else 2.0 ** -22
    assert np.all(np.abs(got_h - want_h) <= tol * np.abs(want_h) + 1e-30)


@pytest.mark.parametrize("name", list(SMALL))
def test_forward_small(name):
    rep = pu.check_forward_against_oracle(SMALL[name])
    print(name, rep)


def test_forward_with_null_biases():
    """Zero biases passed as NULL pointers take the no-bias code paths: same bits as with zero arrays."""
    import torch
    lc = SMALL["bf16_lm"]
    h, w = inputs(lc)
    with_arrays = pu.GpuLayer(lc, h, w).forward()
    with_null = pu.GpuLayer(lc, h, w, drop_zero_biases=True)
    assert all(with_null.w[b] is None for b in ("br1", "br2", "b1", "b2"))
    got = with_null.forward()
    torch.cuda.synchronize()
    for a, b in zip(with_arrays, got):
        assert torch.equal(a, b)
    assert with_null.status() == 0


def test_forward_equals_staged_calls_and_is_deterministic():
    import torch
    lc = SMALL["bf16_lm"]
    h, w = inputs(lc)
    gpu = pu.GpuLayer(lc, h, w)
    h1, a1, k1, i1, p1 = gpu.forward()
    h2, a2, k2, i2, p2 = gpu.forward()
    idx, p, assigned, _ = gpu.route(want_probs=False)
    kept, offsets, dest, perm, xperm = gpu.dispatch(idx, p)
    h3 = gpu.combine(gpu.expert_ffn(xperm, offsets), dest)
    torch.cuda.synchronize()
    assert torch.equal(h1, h2) and torch.equal(i1, i2) and torch.equal(p1, p2) and torch.equal(a1, a2)
    assert torch.equal(i1, idx) and torch.equal(a1, assigned) and torch.equal(k1, kept)
    # the one-launch forward and the chain of staged calls are two evaluations of the same layer (the chain
    # rounds p x to the storage type first): each is graded against the oracle on the ids both picked
    ref = oracle.forward(pu.oracle_config(lc), h, w, forced_idx=idx.cpu().numpy())["h_out"]
    pu.assert_outputs_close(tensors.to_numpy_f32(h1), ref, lc.dtype, what="forward")
    pu.assert_outputs_close(tensors.to_numpy_f32(h3), ref, lc.dtype, what="staged chain")


def test_empty_batch():
    import torch
    lc = C["cfg1"].with_tokens(0)
    h, w = inputs(lc)
    gpu = pu.GpuLayer(lc, h, w)
    h_out, assigned, kept, idx, p = gpu.forward()
    torch.cuda.synchronize()
    assert h_out.numel() == 0 and not assigned.any() and not kept.any()


def test_forward_host_matches_forward():
    import torch
    lc = SMALL["bf16_lm"]
    h, w = inputs(lc)
    gpu = pu.GpuLayer(lc, h, w)
    h_dev = gpu.forward()[0]
    h_host = tensors.to_torch(h, lc.dtype, "cpu", pin=True)
    out_host = torch.empty_like(h_host).pin_memory()
    binding.slicemoe_forward_host(gpu.cfg, gpu.w, h_host, out_host, gpu.ws)
    torch.cuda.synchronize()
    assert torch.equal(out_host, h_dev.cpu())


def test_forward_host_pipelined_in_chunks():
    """From 2048 tokens on (no capacity limit) the host-buffer forward runs in four chunks with
    overlapping copies: same bits as the device forward, counts summed over the chunks, and the
    caller's stream alone orders the result."""
    import torch
    lc = C["cfg1"].with_tokens(2048 + 77)            # ragged last chunk
    h, w = inputs(lc)
    gpu = pu.GpuLayer(lc, h, w)
    h_dev, assigned_dev, kept_dev, _, _ = gpu.forward()
    h_host = tensors.to_torch(h, lc.dtype, "cpu", pin=True)
    out_host = torch.zeros_like(h_host).pin_memory()
    assigned = torch.full((lc.E,), -5, dtype=torch.int32, device="cuda")
    kept = torch.full((lc.E,), -5, dtype=torch.int32, device="cuda")
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        for _ in range(3):                           # back-to-back calls reuse the staging buffers
            binding.slicemoe_forward_host(gpu.cfg, gpu.w, h_host, out_host, gpu.ws, assigned, kept)
    s.synchronize()                                  # only the caller's stream
    assert torch.equal(out_host, h_dev.cpu())
    assert torch.equal(assigned, assigned_dev) and torch.equal(kept, kept_dev)
    assert gpu.status() == 0


def test_forward_host_with_capacity_is_not_chunked():
    """With a capacity limit the drop order spans the whole batch: one forward, same result."""
    import torch
    lc = LC("hostcap", T=2304, d=256, S=4, E=16, k=2, F=256, capacity=300)
    h, w = inputs(lc)
    gpu = pu.GpuLayer(lc, h, w)
    h_dev, _, kept_dev, _, _ = gpu.forward()
    h_host = tensors.to_torch(h, lc.dtype, "cpu", pin=True)
    out_host = torch.zeros_like(h_host).pin_memory()
    kept = torch.zeros((lc.E,), dtype=torch.int32, device="cuda")
    binding.slicemoe_forward_host(gpu.cfg, gpu.w, h_host, out_host, gpu.ws, None, kept)
    torch.cuda.synchronize()
    assert torch.equal(out_host, h_dev.cpu()) and torch.equal(kept, kept_dev)
    assert int(kept.max()) == 300                    # the limit binds, so chunking would have changed the result


def test_forward_host_with_logit_noise_is_not_chunked():
    """Section 3.3's logit noise is drawn per global row number: the host-buffer forward of a batch large
    enough for the chunked pipeline must pick the same experts and give the same bits as the device forward."""
    import torch
    lc = LC("hostnoise", T=2048 + 130, d=512, S=8, E=16, k=2, F=256, noise_sigma=0.5, noise_seed=99)
    h, w = inputs(lc)
    gpu = pu.GpuLayer(lc, h, w)
    h_dev, assigned_dev, kept_dev, _, _ = gpu.forward()
    quiet = pu.GpuLayer(dataclasses.replace(lc, noise_sigma=0.0), h, w)
    assert not torch.equal(quiet.forward()[1], assigned_dev)          # the noise really moves the routing
    h_host = tensors.to_torch(h, lc.dtype, "cpu", pin=True)
    out_host = torch.zeros_like(h_host).pin_memory()
    assigned = torch.zeros((lc.E,), dtype=torch.int32, device="cuda")
    kept = torch.zeros((lc.E,), dtype=torch.int32, device="cuda")
    binding.slicemoe_forward_host(gpu.cfg, gpu.w, h_host, out_host, gpu.ws, assigned, kept)
    torch.cuda.synchronize()
    assert torch.equal(out_host, h_dev.cpu())
    assert torch.equal(assigned, assigned_dev) and torch.equal(kept, kept_dev)


def test_profiled_forward_records_stage_times():
    import torch
    lc = SMALL["bf16_lm"]
    h, w = inputs(lc)
    gpu = pu.GpuLayer(lc, h, w)
    ev = binding.StageEvents()
    h_out = gpu.empty((lc.T, lc.d), gpu.tdtype)
    before = binding.slicemoe_launch_count()
    binding.slicemoe_forward_profiled(gpu.cfg, gpu.w, gpu.h, h_out, gpu.ws, ev)
    ms = ev.stage_ms()
    # route, dispatch and the expert kernel always run; with k <= 2 on the tensor-core path the
    # combine step is folded into the expert kernel and its stage is empty
    assert len(ms) == 4 and all(m > 0 for m in ms[:3]) and ms[3] >= 0
    assert binding.slicemoe_launch_count() - before >= 3
    assert torch.equal(h_out, gpu.forward()[0])


@pytest.mark.parametrize("name", ["bf16_lm", "bf16_skew_cap", "bf16_decode", "bf16_single_row", "bf16_k3", "f32_cfg0",
                                  "bf16_paper_slice96", "bf16_paper_slice48", "bf16_paper_slice192", "bf16_e8"])
def test_forward_launch_count_and_status(name):
    """Supported bf16 shapes with k <= 2 run the whole forward as one launch (slices of 192 / 256 elements with a
    256-wide router: the router, whose weights fill the shared memory, and one launch for the rest); the others
    one launch per step.  Either way the status word stays clear and repeated calls on two workspaces give the same bits."""
    import torch
    lc = SMALL[name]
    h, w = inputs(lc)
    gpu = pu.GpuLayer(lc, h, w)
    gpu2 = pu.GpuLayer(lc, h, w)
    first = gpu.forward()
    before = binding.slicemoe_launch_count()
    again = gpu.forward()
    launches = binding.slicemoe_launch_count() - before
    other = gpu2.forward()
    torch.cuda.synchronize()
    one_launch = lc.dtype == "bf16" and lc.k <= 2 and lc.ds in (48, 64, 96, 128, 192, 256) and lc.E in (8, 16, 32, 64)
    wide_router = one_launch and lc.ds in (192, 256) and lc.Hr == 256
    assert launches == (2 if wide_router else 1) if one_launch else launches >= 3
    assert gpu.status() == 0 and gpu2.status() == 0
    for a, b, c in zip(first, again, other):
        assert torch.equal(a, b) and torch.equal(a, c)


def test_forward_back_to_back_on_two_streams():
    """Launches of the single-kernel forward queued on two streams share the device's grid-barrier
    words; each must still see its own barriers complete."""
    import torch
    lc = SMALL["bf16_lm"]
    h, w = inputs(lc)
    a, b = pu.GpuLayer(lc, h, w), pu.GpuLayer(lc, h, w)
    want = a.forward()[0].clone()
    torch.cuda.synchronize()
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    outs = []
    for i in range(6):
        with torch.cuda.stream(s1 if i % 2 == 0 else s2):
            outs.append((a if i % 2 == 0 else b).forward()[0].clone())
    torch.cuda.synchronize()
    assert a.status() == 0 and b.status() == 0
    for o in outs:
        assert torch.equal(o, want)


def test_dispatch_drops_out_of_range_ids():
    import torch
    lc = SMALL["bf16_lm"]
    h, w = inputs(lc)
    gpu = pu.GpuLayer(lc, h, w)
    rng = np.random.default_rng(3)
    idx_np = rng.integers(0, lc.E, (lc.N, lc.k)).astype(np.int32)
    idx_np[::7, 0] = -1
    idx_np[::11, 1] = lc.E + 3
    p = torch.rand((lc.N, lc.k), device="cuda")
    kept, offsets, dest, perm, xperm = gpu.dispatch(torch.from_numpy(idx_np).cuda(), p)
    torch.cuda.synchronize()
    valid = (idx_np >= 0) & (idx_np < lc.E)
    d = dest.cpu().numpy()
    assert np.all(d[~valid] == -1) and np.all(d[valid] >= 0)
    np.testing.assert_array_equal(kept.cpu().numpy(), np.bincount(idx_np[valid], minlength=lc.E))


# ---- full-size workloads, in the launch configuration the bench times ------------------------

def test_forward_full_cfg1():
    rep = pu.check_forward_against_oracle(C["cfg1"])
    print("cfg1", rep)


def test_forward_full_cfg4_decode():
    rep = pu.check_forward_against_oracle(C["cfg4"])
    print("cfg4", rep)


def test_forward_token_level_decode():
    """The decode batch as a token-level MoE (S = 1: slices are whole tokens, 4096-wide rows) with the
    slice experts' hidden width: the comparison workload beside cfg4, on the CUDA-core kernels."""
    rep = pu.check_forward_against_oracle(C["cfg4_token"])
    print("cfg4_token", rep)


def test_forward_cfg4b_same_E_token_moe():
    """The decode batch as a token-level MoE with whole-token experts (S = 1, FFN 4096 -> 16384 -> 4096, E = 64,
    k = 2): 17 GB of expert weights, drawn and uploaded one expert at a time; only the experts that the
    router picks are drawn (the others are never read).  Routing is graded on all 128 rows, every element of
    h' against the oracle's Eq. 1 / expert FFN / sum run expert by expert on the ids the GPU picked."""
    import dataclasses
    import torch
    lc = C["cfg4b"]
    cfg = tensors.config_from_synth(lc)
    h_np = synth.make_tokens(lc)
    wr = synth.make_router_weights(lc)
    ocfg = pu.oracle_config(lc)
    w = tensors.weights_to_torch(wr, lc.dtype, drop_zero_biases=True)
    w["W1"] = torch.empty((lc.E, lc.F, lc.ds), dtype=torch.bfloat16, device="cuda")
    w["W2"] = torch.empty((lc.E, lc.ds, lc.F), dtype=torch.bfloat16, device="cuda")
    w["b1"] = w["b2"] = None
    h = tensors.to_torch(h_np, lc.dtype)
    ws = binding.alloc_workspace(cfg)
    idx = torch.empty((lc.N, lc.k), dtype=torch.int32, device="cuda")
    p = torch.empty((lc.N, lc.k), dtype=torch.float32, device="cuda")
    assigned = torch.empty((lc.E,), dtype=torch.int32, device="cuda")
    binding.slicemoe_route(cfg, w, h, idx, p, assigned, ws=ws)
    torch.cuda.synchronize()
    idx_np = idx.cpu().numpy()
    ref_route = oracle.route(ocfg, h_np, wr)
    excluded = pu.check_routing(ref_route["probs"], ref_route["gap"], ref_route["topk_idx"], idx_np,
                                p.cpu().numpy().astype(np.float64))
    # the experts the router picked: drawn, uploaded, and used by the oracle, one at a time
    touched = sorted(set(int(e) for e in idx_np.ravel()))
    ref = np.zeros((lc.N, lc.ds), np.float64)
    ocfg1 = dataclasses.replace(ocfg, E=1, k=1)
    x = np.asarray(h_np, np.float64).reshape(lc.N, lc.ds)
    zeros_b1, zeros_b2 = np.zeros((1, lc.F)), np.zeros((1, lc.ds))
    for e in touched:
        we = synth.make_expert_weights(lc, e)
        w["W1"][e].copy_(tensors.to_torch(we["W1"], lc.dtype))
        w["W2"][e].copy_(tensors.to_torch(we["W2"], lc.dtype))
        rows, js = np.nonzero(idx_np == e)
        gates = ref_route["probs"][rows, e]                                  # Eq. 1: the oracle's probability of the id
        xt = gates[:, None] * x[rows]
        y = oracle.expert_ffn(ocfg1, xt, np.array([0, len(rows)]),
                              dict(W1=we["W1"][None], b1=zeros_b1, W2=we["W2"][None], b2=zeros_b2))
        np.add.at(ref, rows, y)
        del we
    out = torch.empty_like(h)
    binding.slicemoe_forward(cfg, w, h, out, ws, topk_idx=idx, topk_p=p, assigned=assigned)
    torch.cuda.synchronize()
    assert binding.slicemoe_last_status(ws) == 0
    assert np.array_equal(idx.cpu().numpy(), idx_np)
    errs = pu.assert_outputs_close(tensors.to_numpy_f32(out).reshape(lc.N, lc.ds), ref, lc.dtype)
    print("cfg4b", dict(touched=len(touched), excluded=excluded, **errs))


def test_forward_full_cfg3_capacity():
    for name in ("cfg3", "cfg3b"):
        rep = pu.check_forward_against_oracle(C[name], sample_rows=16384)
        print(name, rep)


def test_forward_paper_model_shape():
    """The paper's own layer (d = 768, S = 8: 96-wide slices, E = 16, k = 2, F = 4 ds) at a batch of a
    few thousand tokens: runs on the 128-wide tensor-core instantiation with zero-filled columns."""
    lc = LC("paper768", T=3000, d=768, S=8, E=16, k=2, F=384)
    rep = pu.check_forward_against_oracle(lc, sample_rows=4096)
    print("paper768", rep)
    import torch
    h, w = inputs(lc)
    gpu = pu.GpuLayer(lc, h, w)
    before = binding.slicemoe_launch_count()
    gpu.forward()
    torch.cuda.synchronize()
    assert binding.slicemoe_launch_count() - before == 1          # the single-kernel path, not the CUDA-core one


def test_forward_full_cfg2_sampled_rows():
    rep = pu.check_forward_against_oracle(C["cfg2"], sample_rows=65536)
    print("cfg2", rep)


@pytest.mark.parametrize("T,E,k,init", [
    (9485, 16, 2, "normal"),     # 593 router tiles: five per CTA (list groups of 4 + 1), ragged last tile, ragged expert tiles
    (1200, 8, 1, "normal"),      # 75 tiles: one per CTA, half of the CTAs idle; E = 8 on the 16-wide router, k = 1
    (21312, 32, 2, "normal"),    # nine tiles per CTA (groups of 4 + 4 + 1), E = 32: the largest expert count with lists
    (4100, 16, 2, "kaiming"),    # real biases on all four Linears through the bias paths of both passes
])
def test_forward_64wide_list_dispatch_shapes(T, E, k, init):
    """The one-launch forward of 64-wide slices, whose router fills the per-expert lists in groups of tiles:
    group boundaries, CTAs without tiles, ragged tails and both bias paths against the oracle (routing and counts
    on every row, outputs on sampled rows)."""
    import torch
    lc = dataclasses.replace(C["cfg1"], name=f"w64_T{T}_E{E}_k{k}_{init}", T=T, E=E, k=k, init=init)
    rep = pu.check_forward_against_oracle(lc, sample_rows=8192, one_ulp_of_element=(init == "kaiming"))
    print(lc.name, rep)
    h_np, w_np = synth.make_layer_inputs(lc)
    gpu = pu.GpuLayer(lc, h_np, w_np)
    before = binding.slicemoe_launch_count()
    first = gpu.forward()
    torch.cuda.synchronize()
    assert binding.slicemoe_launch_count() - before == 1          # the single-kernel path
    # the order of an expert's list varies from run to run (reservations by atomics); the result must not
    again = gpu.forward()
    torch.cuda.synchronize()
    for a, b in zip(first, again):
        assert torch.equal(a, b)


def test_forward_random_wide_slice_shapes():
    """Sixteen seeded random shapes with slices of 96 to 256 elements (E, k, S, F, batch size, activation, bias
    init and capacity limit drawn at random): the forward against the oracle, the staged route without the
    probability matrix against the oracle's routing, and two forwards on the same workspace bit for bit.  Covers
    the router with resident weights, its hand-over to the single kernel and the split expert tiles on shapes
    nobody picked by hand."""
    import torch
    rng = np.random.default_rng(20251004286)
    for i in range(16):
        E = int(rng.choice([8, 16, 32, 64]))
        k = int(rng.choice([1, 1, 2]))
        ds = int(rng.choice([96, 128, 192, 256, 256]))
        S = int(rng.choice([1, 2, 4]))
        F = int(rng.choice([2, 4])) * ds
        T = max(1, int(rng.choice([1, 17, 129, 500, 1111, 2500, 6000, 12000])) // S)
        init = str(rng.choice(["normal", "kaiming"]))
        act = int(rng.choice([0, 1]))
        cap = int(rng.choice([0, 0, 1])) * max(1, int(1.25 * T * S * k / E) // int(rng.choice([1, 4, 40])))
        lc = LC(f"rw{i}", T=T, d=ds * S, S=S, E=E, k=k, F=F, act=act, init=init, capacity=cap)
        rep = pu.check_forward_against_oracle(lc, seed=int(rng.integers(1 << 30)), sample_rows=2048,
                                              one_ulp_of_element=True)
        h, w = inputs(lc)
        gpu = pu.GpuLayer(lc, h, w)
        idx, p, _, _ = gpu.route(want_probs=False)
        torch.cuda.synchronize()
        ref = oracle.route(pu.oracle_config(lc), h, w)
        pu.check_routing(ref["probs"], ref["gap"], ref["topk_idx"], idx.cpu().numpy(), p.cpu().numpy().astype(np.float64))
        a, b = gpu.forward(), gpu.forward()
        torch.cuda.synchronize()
        assert all(torch.equal(x, y) for x, y in zip(a, b)) and gpu.status() == 0
        print(lc.name, dict(T=T, S=S, ds=ds, E=E, k=k, F=F, act=act, init=init, capacity=cap), rep)

