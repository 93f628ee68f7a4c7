"""Randomised shapes through the forward call, against the oracle: slice widths of the tensor-core
set and others, 8 to 64 experts, k = 1..3, ragged token counts, hard capacities, both activations,
both weight recipes, sharp and flat routers.  Seeded, so a failure names its shape."""
import random

import pytest

from paper_2510_04286_b200 import synth

import parity_util as pu

LC = synth.LayerConfig


def _shape(it, rnd):
    ds = rnd.choice([24, 48, 64, 64, 96, 128, 192, 256])
    S = rnd.choice([1, 2, 4, 8])
    E = rnd.choice([8, 16, 32, 64])
    k = rnd.choice([1, 2, 2, 3])
    T = rnd.choice([1, 3, 17, 64, 100, 257, 600, 1500])
    cap = 0
    if rnd.random() < 0.3:
        cap = max(1, int(rnd.uniform(0.3, 1.5) * T * S * k / E))
    return LC(f"rand{it}", T=T, d=ds * S, S=S, E=E, k=k, F=64 * rnd.randint(2, 12), Hr=rnd.choice([128, 256, 512]),
              act=rnd.choice([0, 1]), init=rnd.choice(["normal", "kaiming"]), capacity=cap,
              wr2_gain=rnd.choice([1.0, 1.0, 30.0]))


@pytest.mark.gpu
@pytest.mark.parametrize("block", range(4))
def test_random_shapes(block):
    rnd = random.Random(1000 + block)
    for it in range(10):
        lc = _shape(10 * block + it, rnd)
        try:
            rep = pu.check_forward_against_oracle(lc, seed=it, one_ulp_of_element=True)
        except AssertionError as ex:
            raise AssertionError(f"{lc}: {ex}") from ex
        assert rep["rel_fro"] <= 6e-3, (lc, rep)
