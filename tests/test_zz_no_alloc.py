"""The allocation-free dispatch entry point against the ordinary one.

slicemoe_dispatch_static serves hosts that cannot obtain device memory when they need a dispatch
(a plugin inside another runtime's arena, a serving loop with all memory fixed at start-up): its
histogram table is a fixed array inside the library instead of a caller workspace.  It must give
bit-identical results to slicemoe_dispatch, also on a second call that finds the first call's
leftovers in the shared array.  This file is collected last on purpose."""
import ctypes

import numpy as np
import pytest

from paper_2510_04286_b200 import binding, synth, tensors


def _outputs(torch, cfg, tdtype):
    return dict(kept=torch.full((cfg.E,), -7, dtype=torch.int32, device="cuda"),
                offsets=torch.full((cfg.E + 1,), -7, dtype=torch.int32, device="cuda"),
                dest=torch.full((cfg.N, cfg.k), -7, dtype=torch.int32, device="cuda"),
                perm=torch.full((cfg.R,), -7, dtype=torch.int32, device="cuda"),
                xperm=torch.zeros((cfg.R, cfg.ds), dtype=tdtype, device="cuda"))


@pytest.mark.gpu
def test_static_dispatch_matches_workspace_dispatch_twice():
    import torch
    # two different problems back to back: the second call sees the table the first one left
    cases = [synth.CONFIGS["cfg1"].with_tokens(700), synth.CONFIGS["cfg3b"].with_tokens(300)]
    for lc in cases:
        cfg = tensors.config_from_synth(lc)
        tdtype = binding.torch_dtype(cfg)
        rng = np.random.default_rng(11)
        h = tensors.to_torch(synth.make_tokens(lc), lc.dtype)
        # k distinct experts per row, skewed so that the capacity case really drops pairs
        scores = rng.random((lc.N, lc.E)) * np.linspace(2.0, 0.5, lc.E)
        idx = torch.from_numpy(np.argsort(-scores, axis=1)[:, :lc.k].astype(np.int32)).cuda()
        p = torch.from_numpy(rng.random((lc.N, lc.k)).astype(np.float32)).cuda()
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
            for name in ref:                       # integer results and copied rows: bit-exact
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
