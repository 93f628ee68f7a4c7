"""Plumbing between the seeded numpy inputs and torch device tensors (no layer arithmetic)."""
from __future__ import annotations

import numpy as np

from . import binding, synth


def config_from_synth(lc: synth.LayerConfig) -> binding.Config:
    return binding.Config(T=lc.T, d=lc.d, S=lc.S, E=lc.E, k=lc.k, F=lc.F, Hr=lc.Hr,
                          dtype=binding.BF16 if lc.dtype == "bf16" else binding.F32,
                          act=lc.act, capacity=lc.capacity, temperature=lc.temperature,
                          noise_sigma=lc.noise_sigma, noise_seed=lc.noise_seed)


def to_torch(arr: np.ndarray, dtype: str, device="cuda", pin=False):
    """A float32 numpy array of stored values -> a torch tensor of the storage dtype (exact)."""
    import torch
    arr = np.ascontiguousarray(arr, dtype=np.float32)
    if dtype == "bf16":
        t = torch.from_numpy(synth.bf16_bits(arr).view(np.int16)).view(torch.bfloat16)
    else:
        t = torch.from_numpy(arr)
    if device == "cpu":
        return t.pin_memory() if pin else t
    return t.to(device)


def weights_to_torch(w: dict, dtype: str, device="cuda", drop_zero_biases=False) -> dict:
    out = {}
    for name, arr in w.items():
        if drop_zero_biases and name.startswith("b") and not np.any(arr):
            out[name] = None
        else:
            out[name] = to_torch(arr, dtype, device)
    return out


def to_numpy_f32(t) -> np.ndarray:
    import torch
    return t.detach().to(torch.float32).cpu().numpy()
