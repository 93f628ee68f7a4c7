"""Thin ctypes binding of libslicemoe.so (the C ABI declared in include/slicemoe.h).

Argument marshalling only: every step of the layer runs in the library's CUDA kernels.  Torch is
used for device memory and the current stream.  There is no fallback: if the shared library is
missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libslicemoe.so")

BF16, F32 = 0, 1
ACT_RELU, ACT_GELU_TANH = 0, 1
N_STAGE_EVENTS = 5
STAGES = ("route", "dispatch", "expert_ffn", "combine")

EXPORTS = (
    "slicemoe_workspace_bytes", "slicemoe_route", "slicemoe_dispatch", "slicemoe_dispatch_static",
    "slicemoe_expert_ffn",
    "slicemoe_combine", "slicemoe_gate_dropout", "slicemoe_permute_columns", "slicemoe_load_stats", "slicemoe_forward", "slicemoe_forward_host", "slicemoe_forward_profiled",
    "slicemoe_event_create", "slicemoe_event_destroy", "slicemoe_event_elapsed_ms",
    "slicemoe_last_status", "slicemoe_launch_count", "slicemoe_last_cuda_error",
    "slicemoe_status_string", "slicemoe_backward_workspace_bytes", "slicemoe_backward",
)


class SliceMoEError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        msg = _lib().slicemoe_status_string(status).decode()
        detail = _lib().slicemoe_last_cuda_error().decode() if status == 7 else ""
        super().__init__(f"{what}: status {status} ({msg}){' -- ' + detail if detail else ''}")


class _Config(ctypes.Structure):
    _fields_ = [("T", ctypes.c_int32), ("d", ctypes.c_int32), ("S", ctypes.c_int32),
                ("E", ctypes.c_int32), ("k", ctypes.c_int32), ("Hr", ctypes.c_int32),
                ("F", ctypes.c_int32), ("dtype", ctypes.c_int32), ("act", ctypes.c_int32),
                ("capacity", ctypes.c_int64), ("temperature", ctypes.c_float),
                ("noise_sigma", ctypes.c_float), ("noise_seed", ctypes.c_uint64),
                ("train_gates", ctypes.c_int32), ("dropout_rate", ctypes.c_float), ("dropout_seed", ctypes.c_uint64)]


class _Weights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("Wr1", "br1", "Wr2", "br2", "W1", "b1", "W2", "b2")]


@dataclass(frozen=True)
class Config:
    """Shape of one SliceMoE layer (paper notation)."""
    T: int
    d: int
    S: int
    E: int
    k: int
    F: int
    Hr: int = 256
    dtype: int = BF16
    act: int = ACT_GELU_TANH
    capacity: int = 0
    temperature: float = 0.0     # softmax temperature of the router (0 stands for 1)
    noise_sigma: float = 0.0     # std of Gaussian noise on the router logits
    noise_seed: int = 0
    train_gates: int = 0         # forward calls: 1 = Section 3.3's gates (cross-slice dropout) instead of the probabilities
    dropout_rate: float = 0.0
    dropout_seed: int = 0

    @property
    def ds(self):
        return self.d // self.S

    @property
    def N(self):
        return self.T * self.S

    @property
    def R(self):
        return self.T * self.S * self.k

    def c(self) -> _Config:
        return _Config(self.T, self.d, self.S, self.E, self.k, self.Hr, self.F, self.dtype, self.act,
                       self.capacity, self.temperature, self.noise_sigma, self.noise_seed,
                       self.train_gates, self.dropout_rate, self.dropout_seed)


_handle = None


def _lib():
    """Loads libslicemoe.so; raises if it has not been built (no fallback exists)."""
    global _handle
    if _handle is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2510_04286_b200.build`")
        lib = ctypes.CDLL(LIB_PATH)
        for name in EXPORTS:
            getattr(lib, name)  # AttributeError if a declared symbol is not exported
        lib.slicemoe_status_string.restype = ctypes.c_char_p
        lib.slicemoe_last_cuda_error.restype = ctypes.c_char_p
        lib.slicemoe_launch_count.restype = ctypes.c_int64
        _handle = lib
    return _handle


def _ptr(t):
    if t is None:
        return ctypes.c_void_p(None)
    if not t.is_contiguous():
        raise ValueError("tensors passed to the SliceMoE library must be contiguous")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _check(status, what):
    if status != 0:
        raise SliceMoEError(status, what)


def _weights(w: dict) -> _Weights:
    def p(name):
        t = w.get(name)
        return None if t is None else t.data_ptr()
    for name in w:
        if w[name] is not None and not w[name].is_contiguous():
            raise ValueError(f"weight {name} must be contiguous")
    return _Weights(*(p(n) for n in ("Wr1", "br1", "Wr2", "br2", "W1", "b1", "W2", "b2")))


def torch_dtype(cfg: Config):
    import torch
    return torch.bfloat16 if cfg.dtype == BF16 else torch.float32


def slicemoe_workspace_bytes(cfg: Config) -> int:
    out = ctypes.c_size_t(0)
    c = cfg.c()
    _check(_lib().slicemoe_workspace_bytes(ctypes.byref(c), ctypes.byref(out)), "slicemoe_workspace_bytes")
    return int(out.value)


def alloc_workspace(cfg: Config, device="cuda"):
    """A workspace tensor of the size the library asks for (torch's allocator aligns it to 512 B)."""
    import torch
    return torch.empty(slicemoe_workspace_bytes(cfg), dtype=torch.uint8, device=device)


def slicemoe_route(cfg, w, h, topk_idx, topk_p, assigned, probs=None, ws=None, stream=None):
    c, ww = cfg.c(), _weights(w)
    _check(_lib().slicemoe_route(ctypes.byref(c), ctypes.byref(ww), _ptr(h), _ptr(topk_idx), _ptr(topk_p),
                                 _ptr(assigned), _ptr(probs), _ptr(ws), ctypes.c_size_t(ws.numel()),
                                 _stream(stream)), "slicemoe_route")


def slicemoe_dispatch(cfg, h, topk_idx, topk_p, kept, offsets, dest, perm, xperm, ws, stream=None):
    c = cfg.c()
    _check(_lib().slicemoe_dispatch(ctypes.byref(c), _ptr(h), _ptr(topk_idx), _ptr(topk_p), _ptr(kept),
                                    _ptr(offsets), _ptr(dest), _ptr(perm), _ptr(xperm), _ptr(ws),
                                    ctypes.c_size_t(ws.numel()), _stream(stream)), "slicemoe_dispatch")


STATIC_SCRATCH_INTS = 65536


def slicemoe_dispatch_static(cfg, h, topk_idx, topk_p, kept, offsets, dest, perm, xperm, stream=None):
    """slicemoe_dispatch without a workspace, for callers that may not allocate device memory:
    the histogram table sits in a fixed 256 KiB array inside the library.  Calls share that array,
    so do not let two of them overlap on the GPU; problems with
    ceil(R / 2048) * E > STATIC_SCRATCH_INTS are refused (status 10)."""
    c = cfg.c()
    _check(_lib().slicemoe_dispatch_static(ctypes.byref(c), _ptr(h), _ptr(topk_idx), _ptr(topk_p),
                                           _ptr(kept), _ptr(offsets), _ptr(dest), _ptr(perm), _ptr(xperm),
                                           _stream(stream)), "slicemoe_dispatch_static")


def slicemoe_expert_ffn(cfg, w, xperm, offsets, yperm, ws, stream=None):
    c, ww = cfg.c(), _weights(w)
    _check(_lib().slicemoe_expert_ffn(ctypes.byref(c), ctypes.byref(ww), _ptr(xperm), _ptr(offsets),
                                      _ptr(yperm), _ptr(ws), ctypes.c_size_t(ws.numel()), _stream(stream)),
           "slicemoe_expert_ffn")


def slicemoe_combine(cfg, yperm, dest, h_out, stream=None):
    c = cfg.c()
    _check(_lib().slicemoe_combine(ctypes.byref(c), _ptr(yperm), _ptr(dest), _ptr(h_out), _stream(stream)),
           "slicemoe_combine")


def slicemoe_gate_dropout(cfg, topk_p, seed, rate, stream=None):
    """Section 3.3: topk_p (cuda float32 [N, k]) becomes the train-mode gates, in place."""
    c = cfg.c()
    _check(_lib().slicemoe_gate_dropout(ctypes.byref(c), _ptr(topk_p), ctypes.c_uint64(seed), ctypes.c_double(rate),
                                        _stream(stream)), "slicemoe_gate_dropout")


def slicemoe_permute_columns(cfg, src, dst, perm, inverse=False, stream=None):
    """Figure 5's shuffled slices: dst[t, c] = src[t, perm[c]], or with inverse dst[t, perm[c]] = src[t, c]."""
    c = cfg.c()
    _check(_lib().slicemoe_permute_columns(ctypes.byref(c), _ptr(src), _ptr(dst), _ptr(perm),
                                           ctypes.c_int(1 if inverse else 0), _stream(stream)),
           "slicemoe_permute_columns")


def slicemoe_load_stats(counts, alpha, out, stream=None):
    """counts: cuda int32 [E]; out: cuda float64 [2] <- (L_cap of Eq. 2, ELE of Section 4)."""
    _check(_lib().slicemoe_load_stats(_ptr(counts), ctypes.c_int32(counts.numel()), ctypes.c_double(alpha),
                                      _ptr(out), _stream(stream)), "slicemoe_load_stats")


def slicemoe_forward(cfg, w, h, h_out, ws, assigned=None, kept=None, topk_idx=None, topk_p=None,
                     stream=None):
    c, ww = cfg.c(), _weights(w)
    _check(_lib().slicemoe_forward(ctypes.byref(c), ctypes.byref(ww), _ptr(h), _ptr(h_out), _ptr(assigned),
                                   _ptr(kept), _ptr(topk_idx), _ptr(topk_p), _ptr(ws),
                                   ctypes.c_size_t(ws.numel()), _stream(stream)), "slicemoe_forward")


def slicemoe_forward_host(cfg, w, h_host, h_out_host, ws, assigned=None, kept=None, stream=None):
    """h_host / h_out_host are CPU tensors (pinned for asynchronous copies)."""
    c, ww = cfg.c(), _weights(w)
    if h_host.is_cuda or h_out_host.is_cuda:
        raise ValueError("slicemoe_forward_host takes host tensors")
    _check(_lib().slicemoe_forward_host(ctypes.byref(c), ctypes.byref(ww), _ptr(h_host), _ptr(h_out_host),
                                        _ptr(assigned), _ptr(kept), _ptr(ws), ctypes.c_size_t(ws.numel()),
                                        _stream(stream)), "slicemoe_forward_host")


class StageEvents:
    """The CUDA events slicemoe_forward_profiled records at its stage boundaries."""

    def __init__(self):
        self._ev = (ctypes.c_void_p * N_STAGE_EVENTS)()
        for i in range(N_STAGE_EVENTS):
            e = ctypes.c_void_p()
            _check(_lib().slicemoe_event_create(ctypes.byref(e)), "slicemoe_event_create")
            self._ev[i] = e.value

    def stage_ms(self):
        """Milliseconds of (route, dispatch, expert_ffn, combine); waits for the last event."""
        out = []
        for i in range(N_STAGE_EVENTS - 1):
            ms = ctypes.c_float()
            _check(_lib().slicemoe_event_elapsed_ms(ctypes.c_void_p(self._ev[i]), ctypes.c_void_p(self._ev[i + 1]),
                                                    ctypes.byref(ms)), "slicemoe_event_elapsed_ms")
            out.append(ms.value)
        return out

    def close(self):
        for i in range(N_STAGE_EVENTS):
            if self._ev[i]:
                _lib().slicemoe_event_destroy(ctypes.c_void_p(self._ev[i]))
                self._ev[i] = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def slicemoe_forward_profiled(cfg, w, h, h_out, ws, events: StageEvents, assigned=None, kept=None,
                              topk_idx=None, topk_p=None, stream=None):
    c, ww = cfg.c(), _weights(w)
    _check(_lib().slicemoe_forward_profiled(ctypes.byref(c), ctypes.byref(ww), _ptr(h), _ptr(h_out),
                                            _ptr(assigned), _ptr(kept), _ptr(topk_idx), _ptr(topk_p),
                                            _ptr(ws), ctypes.c_size_t(ws.numel()), _stream(stream),
                                            events._ev), "slicemoe_forward_profiled")


class _Grads(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("dWr1", "dbr1", "dWr2", "dbr2", "dW1", "db1", "dW2", "db2")]


def slicemoe_backward_workspace_bytes(cfg: Config) -> int:
    out = ctypes.c_size_t(0)
    c = cfg.c()
    _check(_lib().slicemoe_backward_workspace_bytes(ctypes.byref(c), ctypes.byref(out)),
           "slicemoe_backward_workspace_bytes")
    return int(out.value)


def slicemoe_backward(cfg, w, h, grad_out, topk_idx, topk_p, grad_h, grads: dict, ws, accumulate=False,
                      dropout_gates=False, stream=None):
    """Backward of the layer: grad_h and the fp32 weight gradients in ``grads`` (keys dWr1, dbr1,
    dWr2, dbr2, dW1, db1, dW2, db2; bias entries may be missing) from grad_out = dL/dh'.  With
    ``dropout_gates`` topk_p holds the gates of slicemoe_gate_dropout (Section 3.3)."""
    import torch
    c, ww = cfg.c(), _weights(w)
    for name, t in grads.items():
        if t is not None and (t.dtype != torch.float32 or not t.is_contiguous()):
            raise ValueError(f"gradient {name} must be a contiguous float32 tensor")
    gg = _Grads(*((None if grads.get(n) is None else grads[n].data_ptr())
                  for n in ("dWr1", "dbr1", "dWr2", "dbr2", "dW1", "db1", "dW2", "db2")))
    _check(_lib().slicemoe_backward(ctypes.byref(c), ctypes.byref(ww), _ptr(h), _ptr(grad_out), _ptr(topk_idx),
                                    _ptr(topk_p), _ptr(grad_h), ctypes.byref(gg), ctypes.c_int(int(accumulate)),
                                    ctypes.c_int(int(dropout_gates)), _ptr(ws), ctypes.c_size_t(ws.numel()), _stream(stream)), "slicemoe_backward")


def slicemoe_last_status(ws, stream=None) -> int:
    return int(_lib().slicemoe_last_status(_ptr(ws), _stream(stream)))


def slicemoe_launch_count() -> int:
    return int(_lib().slicemoe_launch_count())


def slicemoe_status_string(status: int) -> str:
    return _lib().slicemoe_status_string(int(status)).decode()
