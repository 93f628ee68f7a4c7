"""Seeded synthetic inputs for the SliceMoE layer forward.

This module only draws random tensors and rounds them to their storage type.
It holds none of the layer's arithmetic (no router, no softmax, no expert FFN),
so the CUDA path and the CPU oracle can both be fed from it without sharing
any code of the method itself.

Every tensor has its own counter-based sub-stream: Philox keyed by
(seed, tensor id).  Values are rounded to the storage dtype (bf16
round-to-nearest-even, or fp32) *before* anyone reads them and are returned as
float32 arrays that hold exactly those stored values.

Shapes follow the paper's notation (Section 3): a token vector h in R^d is cut
into S contiguous slices of ds = d/S; the shared router MLP is
Linear(ds -> H_r) -> ReLU -> Linear(H_r -> E); each of the E experts is a
two-layer FFN ds -> F -> ds; k experts are chosen per slice.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import numpy as np

ACT_RELU = 0
ACT_GELU_TANH = 1

_TENSOR_IDS = {"h": 0, "Wr1": 1, "br1": 2, "Wr2": 3, "br2": 4,
               "W1": 5, "b1": 6, "W2": 7, "b2": 8, "grad_out": 9}


@dataclass(frozen=True)
class LayerConfig:
    """Shape and input recipe of one synthetic workload."""
    name: str
    T: int
    d: int
    S: int
    E: int
    k: int
    F: int
    Hr: int = 256
    dtype: str = "bf16"          # storage type: "bf16" or "f32"
    act: int = ACT_GELU_TANH
    capacity: int = 0            # 0 = unlimited
    init: str = "normal"         # "normal": N(0, 0.02) weights, zero biases
                                 # "kaiming": He-uniform weights, uniform biases
    zipf_s: float = 0.0          # > 0: router output bias 1.5*log(Zipf(s) weight)
    wr2_gain: float = 1.0        # multiplies the std of Wr2 (calibrated-skew variant)
    temperature: float = 0.0     # router softmax temperature (0 stands for 1)
    noise_sigma: float = 0.0     # std of Gaussian noise on the router logits
    noise_seed: int = 0

    @property
    def ds(self) -> int:
        return self.d // self.S

    @property
    def N(self) -> int:
        return self.T * self.S

    @property
    def R(self) -> int:
        return self.T * self.S * self.k

    def with_tokens(self, T: int) -> "LayerConfig":
        cap = self.capacity
        if cap:
            cap = capacity_for(T, self.S, self.k, self.E)
        return replace(self, T=T, capacity=cap)


def capacity_for(T: int, S: int, k: int, E: int, factor: float = 1.25) -> int:
    """Per-expert capacity ceil(factor * T*S*k / E) of the skewed-routing workload."""
    return int(math.ceil(factor * T * S * k / E))


CONFIGS = {
    # Tiny fp32 layer, all four Linears carry biases, ReLU experts.
    "cfg0": LayerConfig("cfg0", T=512, d=256, S=4, E=8, k=2, F=256, dtype="f32",
                        act=ACT_RELU, init="kaiming"),
    # LM-layer shape (batch 32 x seq 512).
    "cfg1": LayerConfig("cfg1", T=16384, d=512, S=8, E=16, k=2, F=256),
    # Wider layer (batch 64 x seq 1024).
    "cfg2": LayerConfig("cfg2", T=65536, d=1024, S=16, E=32, k=2, F=256),
    # Skewed routing with a hard capacity and overflow drop.
    "cfg3": LayerConfig("cfg3", T=32768, d=2048, S=8, E=64, k=1, F=1024,
                        capacity=capacity_for(32768, 8, 1, 64), zipf_s=1.2),
    # Same, with the router's output layer scaled so that data, not only the
    # bias, decides the expert: several experts overflow instead of one.
    "cfg3b": LayerConfig("cfg3b", T=32768, d=2048, S=8, E=64, k=1, F=1024,
                         capacity=capacity_for(32768, 8, 1, 64), zipf_s=1.2,
                         wr2_gain=100.0),
    # Decode-shaped, weight-bandwidth-bound.
    "cfg4": LayerConfig("cfg4", T=128, d=4096, S=32, E=64, k=2, F=512),
    # Same-E token-level MoE comparison (S = 1).
    "cfg4b": LayerConfig("cfg4b", T=128, d=4096, S=1, E=64, k=2, F=16384),
    # Token-level MoE on the decode batch with the slice experts' hidden width (S = 1: slices are whole
    # tokens); 0.5 GB of expert weights, small enough to generate and to grade against the oracle.
    "cfg4_token": LayerConfig("cfg4_token", T=128, d=4096, S=1, E=64, k=2, F=512),
    # The paper's own model (Section 4): d = 768, S = 8 (96-wide slices), E = 16, k = 2; the expert
    # width F = 4 ds follows the other workloads, the batch is 32 sequences of 512 tokens.
    "paper768": LayerConfig("paper768", T=16384, d=768, S=8, E=16, k=2, F=384),
    # the shapes of the paper's slice-count and top-k ablations (Table 2, Table 4) on the same model
    "paper768_S2": LayerConfig("paper768_S2", T=16384, d=768, S=2, E=16, k=2, F=1536),     # CUDA-core kernels
    "paper768_S32": LayerConfig("paper768_S32", T=16384, d=768, S=32, E=16, k=2, F=96),    # CUDA-core kernels
    "paper768_S4": LayerConfig("paper768_S4", T=16384, d=768, S=4, E=16, k=2, F=768),
    "paper768_S16": LayerConfig("paper768_S16", T=16384, d=768, S=16, E=16, k=2, F=192),
    "paper768_k1": LayerConfig("paper768_k1", T=16384, d=768, S=8, E=16, k=1, F=384),
    "paper768_k3": LayerConfig("paper768_k3", T=16384, d=768, S=8, E=16, k=3, F=384),
}


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return rounded.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """The uint16 bit patterns of float32 values that are already bf16-representable."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def round_to_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return round_to_bf16(x)
    if dtype == "f32":
        return np.ascontiguousarray(x, dtype=np.float32)
    raise ValueError(f"unknown storage dtype {dtype!r}")


def _rng(seed: int, tensor: str) -> np.random.Generator:
    key = np.array([seed, _TENSOR_IDS[tensor]], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def _normal(seed, tensor, shape, std, dtype):
    g = _rng(seed, tensor)
    x = g.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return round_to_storage(x, dtype)


def _uniform(seed, tensor, shape, bound, dtype):
    g = _rng(seed, tensor)
    x = g.random(size=shape, dtype=np.float32)
    x = (x * np.float32(2.0) - np.float32(1.0)) * np.float32(bound)
    return round_to_storage(x, dtype)


def zipf_router_bias(E: int, s: float) -> np.ndarray:
    """1.5 * log(w_e) with w_e = (e+1)^-s / sum_j (j+1)^-s (float64)."""
    w = np.arange(1, E + 1, dtype=np.float64) ** (-s)
    w /= w.sum()
    return 1.5 * np.log(w)


def make_tokens(cfg: LayerConfig, seed: int = 0) -> np.ndarray:
    """h[T, d] ~ N(0, 1), rounded to the storage dtype."""
    return _normal(seed, "h", (cfg.T, cfg.d), 1.0, cfg.dtype)


def make_grad_out(cfg: LayerConfig, seed: int = 0) -> np.ndarray:
    """dL/dh'[T, d] ~ N(0, 1) for the backward, rounded to the storage dtype."""
    return _normal(seed, "grad_out", (cfg.T, cfg.d), 1.0, cfg.dtype)


def make_weights(cfg: LayerConfig, seed: int = 0) -> dict:
    """Router and expert weights, nn.Linear layout [out, in] (in contiguous).

    Returns float32 arrays (exact stored values):
      Wr1[Hr, ds], br1[Hr], Wr2[E, Hr], br2[E],
      W1[E, F, ds], b1[E, F], W2[E, ds, F], b2[E, ds].
    """
    ds, Hr, E, F, dt = cfg.ds, cfg.Hr, cfg.E, cfg.F, cfg.dtype
    w = {}
    if cfg.init == "kaiming":
        def wt(name, shape, fan_in):
            return _uniform(seed, name, shape, math.sqrt(6.0 / fan_in), dt)

        def bs(name, shape, fan_in):
            return _uniform(seed, name, shape, 1.0 / math.sqrt(fan_in), dt)

        w["Wr1"] = wt("Wr1", (Hr, ds), ds)
        w["br1"] = bs("br1", (Hr,), ds)
        w["Wr2"] = wt("Wr2", (E, Hr), Hr)
        w["br2"] = bs("br2", (E,), Hr)
        w["W1"] = wt("W1", (E, F, ds), ds)
        w["b1"] = bs("b1", (E, F), ds)
        w["W2"] = wt("W2", (E, ds, F), F)
        w["b2"] = bs("b2", (E, ds), F)
    elif cfg.init == "normal":
        std = 0.02
        w["Wr1"] = _normal(seed, "Wr1", (Hr, ds), std, dt)
        w["br1"] = np.zeros((Hr,), dtype=np.float32)
        w["Wr2"] = _normal(seed, "Wr2", (E, Hr), std * cfg.wr2_gain, dt)
        w["br2"] = np.zeros((E,), dtype=np.float32)
        w["W1"] = _normal(seed, "W1", (E, F, ds), std, dt)
        w["b1"] = np.zeros((E, F), dtype=np.float32)
        w["W2"] = _normal(seed, "W2", (E, ds, F), std, dt)
        w["b2"] = np.zeros((E, ds), dtype=np.float32)
    else:
        raise ValueError(f"unknown init {cfg.init!r}")
    if cfg.zipf_s > 0.0:
        w["br2"] = round_to_storage(zipf_router_bias(E, cfg.zipf_s).astype(np.float32), dt)
    return w


def make_router_weights(cfg: LayerConfig, seed: int = 0) -> dict:
    """Only the router's tensors of make_weights (same streams, same values)."""
    ds, Hr, E, dt = cfg.ds, cfg.Hr, cfg.E, cfg.dtype
    if cfg.init != "normal":
        raise ValueError("make_router_weights: normal init only")
    std = 0.02
    w = {"Wr1": _normal(seed, "Wr1", (Hr, ds), std, dt), "br1": np.zeros((Hr,), dtype=np.float32),
         "Wr2": _normal(seed, "Wr2", (E, Hr), std * cfg.wr2_gain, dt), "br2": np.zeros((E,), dtype=np.float32)}
    if cfg.zipf_s > 0.0:
        w["br2"] = round_to_storage(zipf_router_bias(E, cfg.zipf_s).astype(np.float32), dt)
    return w


def make_expert_weights(cfg: LayerConfig, e: int, seed: int = 0) -> dict:
    """W1[F, ds] and W2[ds, F] of expert ``e`` alone, ~ N(0, 0.02), from sub-streams of their own keyed by
    (seed, tensor, e).  For layers whose expert tensors are too large to draw in one piece (the token-level
    comparison of the decode workload: 17 GB of expert weights): a consumer draws one expert at a time.
    These are NOT the values make_weights puts at index e of its stacked tensors."""
    if cfg.init != "normal":
        raise ValueError("make_expert_weights: normal init only")

    def draw(name, shape):
        key = np.array([seed, _TENSOR_IDS[name] | ((e + 1) << 32)], dtype=np.uint64)
        x = np.random.Generator(np.random.Philox(key=key)).standard_normal(size=shape, dtype=np.float32)
        x *= np.float32(0.02)
        return round_to_storage(x, cfg.dtype)

    return {"W1": draw("W1", (cfg.F, cfg.ds)), "W2": draw("W2", (cfg.ds, cfg.F))}


def make_layer_inputs(cfg: LayerConfig, seed: int = 0):
    """(h, weights) for one workload."""
    return make_tokens(cfg, seed), make_weights(cfg, seed)
