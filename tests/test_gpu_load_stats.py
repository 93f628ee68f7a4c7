"""GPU parity of the routing statistics (Eq. 2's capacity loss, Section 4's ELE) against the oracle."""
import numpy as np
import pytest

import oracle
from paper_2510_04286_b200 import binding, synth

import parity_util as pu

pytestmark = pytest.mark.gpu


def gpu_stats(counts, alpha):
    import torch
    c = torch.from_numpy(np.asarray(counts, dtype=np.int32)).cuda()
    out = torch.full((2,), -7.0, dtype=torch.float64, device="cuda")
    binding.slicemoe_load_stats(c, alpha, out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


CASES = {
    "uniform": ([5] * 16, 0.1),
    "one_hot": ([0, 0, 40, 0], 0.05),
    "skewed": ([1000, 10, 3, 0, 0, 7, 250, 1], 0.2),
    "single_expert": ([12], 0.1),
    "nothing_routed": ([0] * 8, 0.1),
    "wide": (list(np.random.default_rng(5).integers(0, 10 ** 6, 200)), 0.01),
    "large_counts": ([2 ** 31 - 1, 2 ** 31 - 1, 1, 0, 17], 0.1),
}


@pytest.mark.parametrize("name", list(CASES))
def test_load_stats_matches_oracle(name):
    counts, alpha = CASES[name]
    got = gpu_stats(counts, alpha)
    l_cap, ele = oracle.load_stats(np.asarray(counts, dtype=np.int64), alpha)
    # fp64 on both sides; only the summation order differs
    assert got[0] == pytest.approx(l_cap, rel=1e-12, abs=1e-15)
    assert got[1] == pytest.approx(ele, rel=1e-12, abs=1e-15)


def test_load_stats_closed_forms():
    assert gpu_stats([9] * 32, 0.1) == pytest.approx([0.0, 1.0], abs=1e-14)     # balance: Eq. 2 = 0, ELE = 1
    one_hot = gpu_stats([0, 64, 0, 0], 1.0)
    assert one_hot[1] == pytest.approx(0.0, abs=1e-14)                           # all on one expert: ELE = 0
    assert one_hot[0] == pytest.approx(3.0, rel=1e-13)                           # CV^2 of (0, 64, 0, 0) = E - 1


def test_load_stats_of_a_forward():
    """The counts the forward writes are the input the statistics are meant for."""
    import torch
    lc = synth.CONFIGS["cfg1"].with_tokens(333)
    h, w = synth.make_layer_inputs(lc, 0)
    gpu = pu.GpuLayer(lc, h, w)
    _, assigned, kept, _, _ = gpu.forward()
    out = torch.empty(2, dtype=torch.float64, device="cuda")
    binding.slicemoe_load_stats(assigned, 0.1, out)
    torch.cuda.synchronize()
    l_cap, ele = oracle.load_stats(assigned.cpu().numpy().astype(np.int64), 0.1)
    assert out.cpu().numpy() == pytest.approx([l_cap, ele], rel=1e-12)
    assert 0.0 < ele <= 1.0


def test_load_stats_rejects_bad_arguments():
    import torch
    c = torch.zeros(4, dtype=torch.int32, device="cuda")
    out = torch.zeros(2, dtype=torch.float64, device="cuda")
    with pytest.raises(binding.SliceMoEError):
        binding.slicemoe_load_stats(c, 0.1, None)
    with pytest.raises(binding.SliceMoEError):
        binding._check(binding._lib().slicemoe_load_stats(binding._ptr(c), 0, binding.ctypes.c_double(0.1),
                                                          binding._ptr(out), binding._stream()), "E = 0")
