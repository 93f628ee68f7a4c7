"""ctypes front end of the fp64 CPU oracle (``slicemoe_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the bench's
CPU-baseline leg may import this package; the product path never does, and
this package imports nothing of the CUDA library.

All tensors cross as float64 / int32 / int64 numpy arrays.  Stored bf16 or
fp32 values widen to float64 exactly, so the oracle sees the very numbers the
GPU reads and differs from it only by the GPU's own arithmetic.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "slicemoe_oracle.c")
_LIB = os.path.join(_HERE, "libslicemoe_oracle.so")

ACT_RELU = 0
ACT_GELU_TANH = 1


class _Cfg(ctypes.Structure):
    _fields_ = [("T", ctypes.c_int32), ("d", ctypes.c_int32), ("S", ctypes.c_int32),
                ("E", ctypes.c_int32), ("k", ctypes.c_int32), ("Hr", ctypes.c_int32),
                ("F", ctypes.c_int32), ("act", ctypes.c_int32), ("capacity", ctypes.c_int64),
                ("temperature", ctypes.c_double), ("noise_sigma", ctypes.c_double),
                ("noise_seed", ctypes.c_uint64)]


@dataclass(frozen=True)
class OracleConfig:
    T: int
    d: int
    S: int
    E: int
    k: int
    Hr: int
    F: int
    act: int = ACT_RELU
    capacity: int = 0
    temperature: float = 0.0    # router softmax temperature (0 stands for 1)
    noise_sigma: float = 0.0    # std of Gaussian noise on the router logits
    noise_seed: int = 0

    @property
    def ds(self):
        return self.d // self.S

    @property
    def N(self):
        return self.T * self.S

    @property
    def R(self):
        return self.T * self.S * self.k

    def c(self) -> _Cfg:
        return _Cfg(self.T, self.d, self.S, self.E, self.k, self.Hr, self.F, self.act, self.capacity,
                    self.temperature, self.noise_sigma, self.noise_seed)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, OpenMP over rows) if it is stale."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
           "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.slicemoe_oracle_threads.restype = ctypes.c_int
    return _lib


def threads() -> int:
    """Number of host threads the oracle's row loops use."""
    return int(_load().slicemoe_oracle_threads())


def _f64(a, shape=None):
    if a is None:
        return None
    a = np.ascontiguousarray(a, dtype=np.float64)
    if shape is not None and a.size != int(np.prod(shape)):
        raise ValueError(f"expected {shape}, got {a.shape}")
    return a


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check(rc, what):
    if rc != 0:
        raise RuntimeError(f"{what} failed with oracle status {rc}")


def _router_weights(cfg: OracleConfig, w: dict):
    """The router's tensors alone, widened to float64 (the route call reads nothing else)."""
    return dict(
        Wr1=_f64(w["Wr1"], (cfg.Hr, cfg.ds)), br1=_f64(w.get("br1"), (cfg.Hr,)),
        Wr2=_f64(w["Wr2"], (cfg.E, cfg.Hr)), br2=_f64(w.get("br2"), (cfg.E,)))


def _expert_weights(cfg: OracleConfig, w: dict):
    """The experts' tensors alone, widened to float64 (the expert_ffn call reads nothing else)."""
    return dict(
        W1=_f64(w["W1"], (cfg.E, cfg.F, cfg.ds)), b1=_f64(w.get("b1"), (cfg.E, cfg.F)),
        W2=_f64(w["W2"], (cfg.E, cfg.ds, cfg.F)), b2=_f64(w.get("b2"), (cfg.E, cfg.ds)))


def _weights(cfg: OracleConfig, w: dict):
    ds = cfg.ds
    return dict(
        Wr1=_f64(w["Wr1"], (cfg.Hr, ds)), br1=_f64(w.get("br1"), (cfg.Hr,)),
        Wr2=_f64(w["Wr2"], (cfg.E, cfg.Hr)), br2=_f64(w.get("br2"), (cfg.E,)),
        W1=_f64(w["W1"], (cfg.E, cfg.F, ds)), b1=_f64(w.get("b1"), (cfg.E, cfg.F)),
        W2=_f64(w["W2"], (cfg.E, ds, cfg.F)), b2=_f64(w.get("b2"), (cfg.E, ds)))


def route(cfg: OracleConfig, h, w: dict) -> dict:
    """Section 3.1: probabilities, top-k ids (most probable first), their probabilities,
    the gap p_(k) - p_(k+1) and the per-expert assigned counts."""
    lib, c = _load(), cfg.c()
    h = _f64(h, (cfg.T, cfg.d))
    ww = _router_weights(cfg, w)
    probs = np.empty((cfg.N, cfg.E), np.float64)
    idx = np.empty((cfg.N, cfg.k), np.int32)
    pk = np.empty((cfg.N, cfg.k), np.float64)
    gap = np.empty((cfg.N,), np.float64)
    assigned = np.empty((cfg.E,), np.int64)
    _check(lib.slicemoe_oracle_route(ctypes.byref(c), _p(h), _p(ww["Wr1"]), _p(ww["br1"]),
                                     _p(ww["Wr2"]), _p(ww["br2"]), _p(probs), _p(idx), _p(pk),
                                     _p(gap), _p(assigned)), "route")
    return dict(probs=probs, topk_idx=idx, topk_p=pk, gap=gap, assigned=assigned)


def dispatch(cfg: OracleConfig, topk_idx) -> dict:
    """Section 3.4 grouping with the optional hard capacity (stable in (n, j) order)."""
    lib, c = _load(), cfg.c()
    idx = np.ascontiguousarray(topk_idx, dtype=np.int32).reshape(cfg.N, cfg.k)
    assigned = np.empty((cfg.E,), np.int64)
    kept = np.empty((cfg.E,), np.int64)
    offsets = np.empty((cfg.E + 1,), np.int64)
    dest = np.empty((cfg.N, cfg.k), np.int64)
    perm = np.full((max(cfg.R, 1),), -1, np.int64)
    _check(lib.slicemoe_oracle_dispatch(ctypes.byref(c), _p(idx), _p(assigned), _p(kept),
                                        _p(offsets), _p(dest), _p(perm)), "dispatch")
    return dict(assigned=assigned, kept=kept, offsets=offsets, dest=dest,
                perm=perm[:int(offsets[-1])])


def weight_slices(cfg: OracleConfig, h, topk_p, dest, n_kept: int):
    """Eq. 1: xperm[dest(n, j)] = p_j * x_n for every kept pair."""
    lib, c = _load(), cfg.c()
    h = _f64(h, (cfg.T, cfg.d))
    pk = _f64(topk_p, (cfg.N, cfg.k))
    dest = np.ascontiguousarray(dest, dtype=np.int64).reshape(cfg.N, cfg.k)
    xperm = np.zeros((max(n_kept, 1), cfg.ds), np.float64)
    _check(lib.slicemoe_oracle_weight_slices(ctypes.byref(c), _p(h), _p(pk), _p(dest), _p(xperm)),
           "weight_slices")
    return xperm[:n_kept]


def expert_ffn(cfg: OracleConfig, xperm, offsets, w: dict):
    """Section 3.1 / 3.4: each expert's two-layer FFN over its stacked rows."""
    lib, c = _load(), cfg.c()
    offsets = np.ascontiguousarray(offsets, dtype=np.int64)
    n_kept = int(offsets[-1])
    xperm = _f64(xperm, (n_kept, cfg.ds))
    ww = _expert_weights(cfg, w)
    yperm = np.zeros((max(n_kept, 1), cfg.ds), np.float64)
    _check(lib.slicemoe_oracle_expert_ffn(ctypes.byref(c), _p(xperm), _p(offsets), _p(ww["W1"]),
                                          _p(ww["b1"]), _p(ww["W2"]), _p(ww["b2"]), _p(yperm)),
           "expert_ffn")
    return yperm[:n_kept]


def combine(cfg: OracleConfig, yperm, dest):
    """Section 3.1: sum the k outputs of a slice and put it back at its place in h'."""
    lib, c = _load(), cfg.c()
    dest = np.ascontiguousarray(dest, dtype=np.int64).reshape(cfg.N, cfg.k)
    n_rows = int(dest.max()) + 1 if dest.size else 0
    yperm = _f64(yperm)
    if yperm.size < n_rows * cfg.ds:
        raise ValueError("yperm has fewer rows than dest refers to")
    if yperm.size == 0:
        yperm = np.zeros((1, cfg.ds), np.float64)
    h_out = np.empty((cfg.T, cfg.d), np.float64)
    _check(lib.slicemoe_oracle_combine(ctypes.byref(c), _p(yperm), _p(dest), _p(h_out)), "combine")
    return h_out


def forward(cfg: OracleConfig, h, w: dict, forced_idx=None) -> dict:
    """The whole layer; with ``forced_idx[N, k]`` the expert ids are the caller's while the
    gate values stay the router's probabilities of those ids."""
    lib, c = _load(), cfg.c()
    h = _f64(h, (cfg.T, cfg.d))
    ww = _weights(cfg, w)
    forced = None
    if forced_idx is not None:
        forced = np.ascontiguousarray(forced_idx, dtype=np.int32).reshape(cfg.N, cfg.k)
    out = dict(h_out=np.empty((cfg.T, cfg.d), np.float64),
               probs=np.empty((cfg.N, cfg.E), np.float64),
               topk_idx=np.empty((cfg.N, cfg.k), np.int32),
               topk_p=np.empty((cfg.N, cfg.k), np.float64),
               gap=np.empty((cfg.N,), np.float64),
               assigned=np.empty((cfg.E,), np.int64),
               kept=np.empty((cfg.E,), np.int64),
               offsets=np.empty((cfg.E + 1,), np.int64),
               dest=np.empty((cfg.N, cfg.k), np.int64))
    _check(lib.slicemoe_oracle_forward(
        ctypes.byref(c), _p(h), _p(ww["Wr1"]), _p(ww["br1"]), _p(ww["Wr2"]), _p(ww["br2"]),
        _p(ww["W1"]), _p(ww["b1"]), _p(ww["W2"]), _p(ww["b2"]), _p(forced),
        _p(out["h_out"]), _p(out["probs"]), _p(out["topk_idx"]), _p(out["topk_p"]), _p(out["gap"]),
        _p(out["assigned"]), _p(out["kept"]), _p(out["offsets"]), _p(out["dest"])), "forward")
    return out


def rows(cfg: OracleConfig, h, w: dict, row_ids, idx, keep) -> dict:
    """Outputs of the sampled slices ``row_ids`` one by one, with their expert ids ``idx`` and
    keep flags given by the caller (from ``dispatch`` on the full routing)."""
    lib, c = _load(), cfg.c()
    h = _f64(h, (cfg.T, cfg.d))
    ww = _weights(cfg, w)
    row_ids = np.ascontiguousarray(row_ids, dtype=np.int64)
    n = row_ids.size
    idx = np.ascontiguousarray(idx, dtype=np.int32).reshape(n, cfg.k)
    keep = np.ascontiguousarray(keep, dtype=np.int32).reshape(n, cfg.k)
    y = np.empty((n, cfg.ds), np.float64)
    p = np.empty((n, cfg.k), np.float64)
    _check(lib.slicemoe_oracle_rows(
        ctypes.byref(c), _p(h), _p(ww["Wr1"]), _p(ww["br1"]), _p(ww["Wr2"]), _p(ww["br2"]),
        _p(ww["W1"]), _p(ww["b1"]), _p(ww["W2"]), _p(ww["b2"]),
        ctypes.c_int64(n), _p(row_ids), _p(idx), _p(keep), _p(y), _p(p)), "rows")
    return dict(y=y, p=p)


def load_stats(counts, alpha: float = 1.0):
    """(L_cap of Eq. 2, ELE of Section 4) of per-expert counts."""
    lib = _load()
    counts = np.ascontiguousarray(counts, dtype=np.int64)
    l_cap, ele = ctypes.c_double(), ctypes.c_double()
    _check(lib.slicemoe_oracle_load_stats(_p(counts), ctypes.c_int32(counts.size),
                                          ctypes.c_double(alpha), ctypes.byref(l_cap),
                                          ctypes.byref(ele)), "load_stats")
    return l_cap.value, ele.value


def philox4x32(ctr, key):
    """One Philox4x32-10 block: ctr 4 x uint32, key 2 x uint32 -> 4 x uint32."""
    lib = _load()
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib.slicemoe_oracle_philox4x32(_p(c), _p(k), _p(out))
    return out


def gate_dropout(topk_p, seed: int, rate: float):
    """Section 3.3: (gates after cross-slice dropout [N, k], dropped mask [N, k] bool)."""
    lib = _load()
    p = np.ascontiguousarray(topk_p, dtype=np.float64)
    N, k = p.shape
    out = np.empty_like(p)
    dropped = np.zeros((N, k), dtype=np.uint8)
    _check(lib.slicemoe_oracle_gate_dropout(_p(p), ctypes.c_int64(N), ctypes.c_int32(k),
                                            ctypes.c_uint64(seed), ctypes.c_double(rate), _p(out),
                                            _p(dropped)), "gate_dropout")
    return out, dropped.astype(bool)


def logit_noise(seed: int, n: int, e: int) -> float:
    """Figure 6: the standard normal that (times sigma) is added to logit e of row n."""
    lib = _load()
    lib.slicemoe_oracle_logit_noise.restype = ctypes.c_double
    return float(lib.slicemoe_oracle_logit_noise(ctypes.c_uint64(seed), ctypes.c_int64(n), ctypes.c_int32(e)))


def permute_columns(x, perm, inverse: bool = False):
    """Figure 5's shuffled slices, written out element by element:
    out[t, c] = x[t, perm[c]], or with inverse out[t, perm[c]] = x[t, c]."""
    x = np.asarray(x)
    perm = np.asarray(perm, dtype=np.int64)
    T, d = x.shape
    if perm.shape != (d,) or sorted(perm.tolist()) != list(range(d)):
        raise ValueError("perm must be a permutation of the d columns")
    out = np.empty_like(x)
    for c in range(d):
        if inverse:
            out[:, perm[c]] = x[:, c]
        else:
            out[:, c] = x[:, perm[c]]
    return out


def forward_shuffled(cfg: OracleConfig, h, w: dict, perm, forced_idx=None) -> dict:
    """The layer on shuffled slices (Section 5.2): slice s of a token holds columns
    perm[s*ds .. (s+1)*ds - 1] of h, and its result goes back to those columns."""
    res = dict(forward(cfg, permute_columns(_f64(h, (cfg.T, cfg.d)), perm), w, forced_idx=forced_idx))
    res["h_out"] = permute_columns(res["h_out"], perm, inverse=True)
    return res


def backward(cfg: OracleConfig, h, w: dict, grad_out, forced_idx=None, dropped=None) -> dict:
    """Gradients of a scalar loss with respect to the layer's input and weights, given
    ``grad_out`` = dL/dh' (chain rule on the forward of Section 3.1 / Eq. 1; the chosen expert
    ids are constants, the gate p carries the router's gradient).  ``dropped[N, k]`` (the mask of
    ``gate_dropout``) switches the gates to Section 3.3's re-normalised survivors.  Keys: ``dh`` and ``dWr1``,
    ``dbr1``, ``dWr2``, ``dbr2``, ``dW1``, ``db1``, ``dW2``, ``db2`` shaped like the weights."""
    lib, c = _load(), cfg.c()
    h = _f64(h, (cfg.T, cfg.d))
    g = _f64(grad_out, (cfg.T, cfg.d))
    ww = _weights(cfg, w)
    forced = None
    if forced_idx is not None:
        forced = np.ascontiguousarray(forced_idx, dtype=np.int32).reshape(cfg.N, cfg.k)
    mask = None
    if dropped is not None:
        mask = np.ascontiguousarray(dropped, dtype=np.uint8).reshape(cfg.N, cfg.k)
    ds = cfg.ds
    out = dict(dh=np.empty((cfg.T, cfg.d), np.float64),
               dWr1=np.empty((cfg.Hr, ds), np.float64), dbr1=np.empty((cfg.Hr,), np.float64),
               dWr2=np.empty((cfg.E, cfg.Hr), np.float64), dbr2=np.empty((cfg.E,), np.float64),
               dW1=np.empty((cfg.E, cfg.F, ds), np.float64), db1=np.empty((cfg.E, cfg.F), np.float64),
               dW2=np.empty((cfg.E, ds, cfg.F), np.float64), db2=np.empty((cfg.E, ds), np.float64))
    _check(lib.slicemoe_oracle_backward(
        ctypes.byref(c), _p(h), _p(ww["Wr1"]), _p(ww["br1"]), _p(ww["Wr2"]), _p(ww["br2"]),
        _p(ww["W1"]), _p(ww["b1"]), _p(ww["W2"]), _p(ww["b2"]), _p(forced), _p(mask), _p(g),
        _p(out["dh"]), _p(out["dWr1"]), _p(out["dbr1"]), _p(out["dWr2"]), _p(out["dbr2"]),
        _p(out["dW1"]), _p(out["db1"]), _p(out["dW2"]), _p(out["db2"])), "backward")
    return out
