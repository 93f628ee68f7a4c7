"""The allocation-free dispatch entry point against the oracle (and against the ordinary entry point).

slicemoe_dispatch_static serves hosts that cannot obtain device memory when they need a dispatch
(a plugin inside another runtime's arena, a serving loop with all memory fixed at start-up): its
histogram table is a fixed array inside the library instead of a caller workspace.  Its integer
results must equal the oracle's Section 3.4 grouping and its copied rows Eq. 1 rounded once, also on a
second call that finds the first call's leftovers in the shared array; and every output must be
bit-identical to slicemoe_dispatch's.  This file is collected last on purpose."""
import ctypes

import numpy as np
import pytest

import oracle
from paper_2510_04286_b200 import binding, synth, tensors

import parity_util as pu


def _outputs(torch, cfg, tdtype):
    return dict(kept=torch.full((cfg.E,), -7, dtype=torch.int32, device="cuda"),
                offsets=torch.full((cfg.E + 1,), -7, dtype=torch.int32, device="cuda"),
                dest=torch.full((cfg.N, cfg.k), -7, dtype=torch.int32, device="cuda"),
                perm=torch.full((cfg.R,), -7, dtype=torch.int32, device="cuda"),
                xperm=torch.zeros((cfg.R, cfg.ds), dtype=tdtype, device="cuda"))


@pytest.mark.gpu
def test_static_dispatch_matches_oracle_twice():
    import torch
    # two different problems back to back: the second call sees the table the first one left
    cases = [synth.CONFIGS["cfg1"].with_tokens(700), synth.CONFIGS["cfg3b"].with_tokens(300)]
    for lc in cases:
        cfg = tensors.config_from_synth(lc)
        tdtype = binding.torch_dtype(cfg)
        rng = np.random.default_rng(11)
        h_np = synth.make_tokens(lc)
        h = tensors.to_torch(h_np, lc.dtype)
        ocfg = pu.oracle_config(lc)
        # k distinct experts per row, skewed so that the capacity case really drops pairs
        scores = rng.random((lc.N, lc.E)) * np.linspace(2.0, 0.5, lc.E)
        idx_np = np.argsort(-scores, axis=1)[:, :lc.k].astype(np.int32)
        p_np = rng.random((lc.N, lc.k)).astype(np.float32)
        idx, p = torch.from_numpy(idx_np).cuda(), torch.from_numpy(p_np).cuda()
        want = oracle.dispatch(ocfg, idx_np)
        n_kept = int(want["offsets"][-1])
        want_x = oracle.weight_slices(ocfg, h_np, p_np.astype(np.float64), want["dest"], n_kept)
        ws = binding.alloc_workspace(cfg)
        ref = _outputs(torch, cfg, tdtype)
        binding.slicemoe_dispatch(cfg, h, idx, p, ref["kept"], ref["offsets"], ref["dest"], ref["perm"],
                                  ref["xperm"], ws)
        torch.cuda.synchronize()
        for call in range(2):
            got = _outputs(torch, cfg, tdtype)
            binding.slicemoe_dispatch_static(cfg, h, idx, p, got["kept"], got["offsets"], got["dest"],
                                             got["perm"], got["xperm"])
            torch.cuda.synchronize()
            # against the oracle: integer results bit-exact, copied rows Eq. 1 with one rounding to bf16
            for name in ("kept", "offsets", "dest"):
                np.testing.assert_array_equal(got[name].cpu().numpy(), want[name], err_msg=f"{lc.name} call {call}: {name}")
            perm = got["perm"].cpu().numpy()
            np.testing.assert_array_equal(perm[:n_kept], want["perm"], err_msg=f"{lc.name} call {call}: perm")
            assert np.all(perm[n_kept:] == -7)                 # nothing written past the kept rows
            x = tensors.to_numpy_f32(got["xperm"])
            assert np.all(np.abs(x[:n_kept] - want_x) <= 2.0 ** -8 * np.abs(want_x) + 1e-30)
            assert not x[n_kept:].any()
            for name in ref:                       # and the ordinary entry point gives the same bits
                assert torch.equal(got[name], ref[name]), f"{lc.name} call {call}: {name} differs"
        if lc.capacity:
            assert (ref["dest"] < 0).any() and ref["kept"].max().item() == lc.capacity


def test_static_dispatch_refuses_what_its_fixed_scratch_cannot_hold():
    lib = binding._lib()
    # 2^20 tokens * 8 slices * 2 -> 8192 chunks * 16 experts = 131072 ints > 65536
    c = binding.Config(T=1 << 20, d=512, S=8, E=16, k=2, F=256).c()
    fake = ctypes.c_void_p(0x1000)
    rc = lib.slicemoe_dispatch_static(ctypes.byref(c), fake, fake, fake, fake, fake, fake, fake, fake, None)
    assert rc == 10
    assert "fixed scratch" in binding.slicemoe_status_string(rc)
    assert binding.STATIC_SCRATCH_INTS == 65536
